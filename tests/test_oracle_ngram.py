"""Pins of the oracle's prompt-lookup drafter (Section 4.1, lookup range K of Table 3)."""
import numpy as np

from oracle import quasar_oracle as qo


def test_hand_cases():
    #            0  1  2  3  4  5  6  7  8
    h = [5, 6, 7, 8, 9, 5, 6, 7]
    assert qo.ngram_draft(h, 3, 1, 3) == [8, 9, 5]           # "5 6 7" occurred at 0: what followed it
    assert qo.ngram_draft(h, 9, 1, 3) == [8, 9, 5, 6, 7]     # the continuation ends with the sequence
    assert qo.ngram_draft(h, 2, 1, 1) == [8, 9]              # n = 1: the last 7 occurred at 2
    assert qo.ngram_draft([1, 2, 3, 4], 3, 1, 3) == []       # nothing repeats
    assert qo.ngram_draft([7, 7, 7, 7], 2, 1, 2) == [7]      # overlapping occurrence, most recent one: one token follows
    assert qo.ngram_draft([1, 2, 9, 1, 2, 8, 1, 2], 1, 2, 2) == [8]     # most recent of two occurrences
    assert qo.ngram_draft([3, 1, 2, 4, 1, 2], 2, 3, 4) == []            # only a 2-gram repeats, below K_min
    assert qo.ngram_draft([4], 3, 1, 3) == [] and qo.ngram_draft([], 3, 1, 3) == []


def test_longest_match_wins_over_a_more_recent_shorter_one():
    # the last token 2 occurred most recently before "6", but the 2-gram "1 2" occurred before "5"
    h = [1, 2, 5, 0, 2, 6, 1, 2]
    assert qo.ngram_draft(h, 1, 1, 1) == [6]
    assert qo.ngram_draft(h, 1, 1, 2) == [5]


def test_periodic_stream_is_drafted_perfectly():
    rng = np.random.default_rng(0)
    period = list(rng.integers(0, 1000, 11))
    stream = period * 6
    for cut in (25, 40, 57):
        d = qo.ngram_draft(stream[:cut], 7, 1, 4)
        assert d == stream[cut:cut + 7]


def test_against_brute_force_on_random_small_alphabets():
    rng = np.random.default_rng(1)
    for _ in range(300):
        L = int(rng.integers(1, 40))
        h = list(rng.integers(0, 3, L))
        gamma, kmin = int(rng.integers(1, 6)), int(rng.integers(1, 3))
        kmax = kmin + int(rng.integers(0, 3))
        want = []
        for n in range(kmax, kmin - 1, -1):                  # restated from the definition
            if n > L - 1:
                continue
            cands = [s for s in range(0, L - n) if h[s:s + n] == h[L - n:]]
            if cands:
                s = max(cands)
                want = h[s + n:s + n + gamma]
                break
        assert qo.ngram_draft(h, gamma, kmin, kmax) == want
