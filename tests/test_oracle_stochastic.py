"""Pins of the oracle's stochastic acceptance (Section 3.1 Eq. 2-3): closed-form cases and the property the
scheme exists for - the emitted token is distributed as the target distribution, whatever the drafter."""
import numpy as np

from oracle import quasar_oracle as qo


def _logits_of(p):
    return np.log(np.asarray(p, np.float64))


def test_inversion_sampling_closed_forms():
    w = np.array([0.0, 1.0, 0.0, 2.0, 0.0])
    assert [qo.sample_by_inversion(w, u) for u in (0.0, 0.3, 1 / 3 + 1e-9, 0.99)] == [1, 1, 3, 3]
    assert qo.sample_by_inversion(np.array([5.0]), 0.7) == 0
    assert qo.sample_by_inversion(w, np.nextafter(1.0, 0.0)) == 3
    # frequencies follow the weights
    us = (np.arange(6000) + 0.5) / 6000
    counts = np.bincount([qo.sample_by_inversion(np.array([1.0, 2.0, 3.0]), u) for u in us], minlength=3)
    assert list(counts) == [1000, 2000, 3000]


def test_softmax_with_temperature():
    l = np.array([1.0, 2.0, 3.0])
    p = qo.softmax_t(l, 1.0)
    assert np.allclose(p, np.exp(l) / np.exp(l).sum(), rtol=1e-15) and abs(p.sum() - 1) < 1e-15
    assert np.allclose(qo.softmax_t(l, 0.5), qo.softmax_t(2 * l, 1.0), rtol=1e-15)
    assert qo.softmax_t(l, 1e-3).argmax() == 2 and qo.softmax_t(l, 1e-3)[2] > 1 - 1e-12      # T -> 0 is greedy


def test_draft_from_the_target_itself_is_always_accepted():
    """q = p: the ratio of Eq. 2 is 1, every r in [0, 1) accepts, and the bonus comes from the last row."""
    rng = np.random.default_rng(0)
    V, T = 16, 5
    p = rng.dirichlet(np.ones(V), T)
    logits = _logits_of(p)
    tokens = [3] + [int(rng.integers(V)) for _ in range(T - 1)]
    for trial in range(20):
        n, tok = qo.accept_stochastic(logits, tokens, p, 1.0, rng.random(T - 1), 0.5)
        assert n == T - 1
        assert tok == qo.sample_by_inversion(p[T - 1], 0.5)


def test_impossible_draft_is_rejected_and_resampled_from_the_target():
    """The drafter puts all its mass on a token the target gives probability 0: rejected at once, and the
    corrective token is drawn from norm(max(0, p - q)) = p (Eq. 3)."""
    V = 8
    p = np.array([0.5, 0.25, 0.25, 0, 0, 0, 0, 0.0])
    logits = np.where(p > 0, np.log(np.maximum(p, 1e-300)), -1e30)[None, :].repeat(3, 0)
    q = np.zeros((3, V)); q[:, 5] = 1.0
    n, tok = qo.accept_stochastic(logits, [0, 5, 5], q, 1.0, np.array([0.0, 0.0]), 0.6)
    assert n == 0 and tok == 1                     # cdf of p: .5, .75, 1 -> u = .6 falls on token 1
    n, tok = qo.accept_stochastic(logits, [0, 5, 5], None, 1.0, np.array([0.0, 0.0]), 0.8)
    assert n == 0 and tok == 2


def test_point_mass_draft_hand_case():
    """Point-mass drafter on token 1 with p = (.2, .5, .3): accepted iff r < .5 (up to the rounding of the softmax); on rejection the residual is
    (.2, 0, .3) / .5."""
    p = np.array([[0.2, 0.5, 0.3], [0.2, 0.5, 0.3]])
    logits = _logits_of(p)
    assert qo.accept_stochastic(logits, [0, 1], None, 1.0, np.array([0.49]), 0.0) == (1, 0)
    assert qo.accept_stochastic(logits, [0, 1], None, 1.0, np.array([0.49]), 0.21) == (1, 1)     # bonus from p: cdf .2, .7, 1
    assert qo.accept_stochastic(logits, [0, 1], None, 1.0, np.array([0.51]), 0.39) == (0, 0)     # residual cdf .4, .4, 1
    assert qo.accept_stochastic(logits, [0, 1], None, 1.0, np.array([0.51]), 0.41) == (0, 2)


def test_emitted_token_follows_the_target_distribution():
    """The lossless guarantee: with drafts drawn from ANY q, the first emitted token of a step (the accepted
    draft, or the corrective token) is distributed as p.  16-token vocabulary, stratified uniforms."""
    rng = np.random.default_rng(1)
    V = 16
    p = rng.dirichlet(np.ones(V) * 0.7)
    q = rng.dirichlet(np.ones(V) * 0.7)
    logits = _logits_of(np.stack([p, p]))
    n = 120
    grid = (np.arange(n) + 0.5) / n
    counts = np.zeros(V)
    weight = 0.0
    for ud in grid:                                  # the drafter's uniform
        draft = qo.sample_by_inversion(q, ud)
        for ra in grid[::4]:
            for rs in grid[::4]:
                acc, tok = qo.accept_stochastic(logits, [0, draft], np.stack([q, q]), 1.0, np.array([ra]), rs)
                counts[draft if acc == 1 else tok] += 1
                weight += 1
    assert np.abs(counts / weight - p).max() < 0.02
    # and with the point-mass drafter on a fixed token
    counts = np.zeros(V)
    for ra in grid:
        for rs in grid:
            acc, tok = qo.accept_stochastic(logits, [0, 4], None, 1.0, np.array([ra]), rs)
            counts[4 if acc == 1 else tok] += 1
    assert np.abs(counts / n ** 2 - p).max() < 0.01
