"""End-to-end invariants that pin the oracle's verification pass (CPU only, tiny model)."""
import numpy as np
import pytest

import oracle
from oracle import quasar_oracle as qo
from paper_2603_01399_b200 import synth
from tests.common import oracle_model, oracle_greedy_continuation, prefill_oracle


@pytest.fixture(scope="module", params=["tiny", "tiny_qknorm"])
def setup(request):
    shape = synth.SHAPES[request.param]
    model = oracle_model(shape, seed=0, int8=True)
    kv = oracle.new_kv(model, 1, 96)
    toks = synth.uniform_tokens((64,), shape.vocab, synth.sub_seed(2, "tokens"))
    prefill_oracle(model, kv, toks[:63].numpy(), chunk=8)
    return shape, model, kv, int(toks[63])


def _copy(kv):
    return oracle.KVCache(kv.k_bits.copy(), kv.v_bits.copy(), kv.seq_len.copy())


def test_own_greedy_draft_is_fully_accepted(setup):
    shape, model, kv, root = setup
    g = oracle_greedy_continuation(model, kv, root, 5)
    r = oracle.verify(model, _copy(kv), np.array([[root] + g[:4]], np.int32), None, np.array([5], np.int32))
    assert r.accept_len[0] == 4 and r.bonus[0] == g[4]
    assert list(r.accept_path[0]) == [0, 1, 2, 3, 4]
    assert list(r.top1[0]) == g


def test_wrong_draft_is_rejected_where_it_diverges(setup):
    shape, model, kv, root = setup
    g = oracle_greedy_continuation(model, kv, root, 5)
    for cut in range(4):
        d = list(g[:4])
        d[cut] = (d[cut] + 1) % shape.vocab
        r = oracle.verify(model, _copy(kv), np.array([[root] + d], np.int32), None, np.array([5], np.int32))
        assert r.accept_len[0] == cut and r.bonus[0] == g[cut]
        assert 0 <= r.accept_len[0] <= 4


def test_block_verify_equals_row_by_row_decode(setup):
    shape, model, kv, root = setup
    rng = np.random.default_rng(5)
    blk = [root] + [int(t) for t in rng.integers(0, shape.vocab, 4)]
    r = oracle.verify(model, _copy(kv), np.array([blk], np.int32), None, np.array([5], np.int32))
    kv2 = _copy(kv)
    for i, t in enumerate(blk):
        ri = oracle.verify(model, kv2, np.array([[t]], np.int32), None, np.array([1], np.int32))
        assert np.allclose(ri.logits[0, 0], r.logits[0, i], rtol=0, atol=1e-6)
        kv2.seq_len[0] += 1


def test_chain_equals_tree_with_chain_parents_and_is_idempotent(setup):
    shape, model, kv, root = setup
    blk = np.array([[root, 3, 4, 5, 6, 0, 0]], np.int32)          # T_max 7, block_len 5: padding ignored
    bl = np.array([5], np.int32)
    kva, kvb = _copy(kv), _copy(kv)
    ra = oracle.verify(model, kva, blk, None, bl)
    rb = oracle.verify(model, kvb, blk, np.array([[-1, 0, 1, 2, 3, 0, 0]], np.int32), bl)
    assert np.array_equal(ra.logits, rb.logits) and np.array_equal(kva.k_bits, kvb.k_bits)
    rc = oracle.verify(model, kva, blk, None, bl)                  # same cache, no commit in between
    assert np.array_equal(ra.logits, rc.logits) and np.array_equal(kva.seq_len, kv.seq_len)
    assert np.all(ra.logits[0, 5:] == 0)


def test_tree_siblings_do_not_see_each_other(setup):
    shape, model, kv, root = setup
    par = np.array([[-1, 0, 0, 1, 2]], np.int32)
    t1 = np.array([[root, 11, 12, 13, 14]], np.int32)
    t2 = np.array([[root, 11, 99, 13, 77]], np.int32)              # change the other branch only
    bl = np.array([5], np.int32)
    r1 = oracle.verify(model, _copy(kv), t1, par, bl)
    r2 = oracle.verify(model, _copy(kv), t2, par, bl)
    assert np.array_equal(r1.logits[0, [0, 1, 3]], r2.logits[0, [0, 1, 3]])
    assert not np.array_equal(r1.logits[0, 2], r2.logits[0, 2])
    # a branch of a tree gives the logits of the same tokens verified as a chain
    rc = oracle.verify(model, _copy(kv), np.array([[root, 12, 14]], np.int32), None, np.array([3], np.int32))
    assert np.allclose(rc.logits[0], r1.logits[0, [0, 2, 4]], rtol=0, atol=1e-6)


def test_tree_commit_then_verify_equals_chain_prefill(setup):
    shape, model, kv, root = setup
    g = oracle_greedy_continuation(model, kv, root, 3)
    par = np.array([[-1, 0, 0, 1, 2, 4]], np.int32)                # greedy path lives on nodes 2 -> 4 -> 5
    tok = np.array([[root, (g[0] + 1) % shape.vocab, g[0], 5, g[1], (g[2] + 7) % shape.vocab]], np.int32)
    kva = _copy(kv)
    r = oracle.verify(model, kva, tok, par, np.array([6], np.int32))
    assert r.accept_len[0] == 2 and list(r.accept_path[0][:3]) == [0, 2, 4] and r.bonus[0] == g[2]
    oracle.kv_commit(kva, r.accept_len, r.accept_path)
    kvb = _copy(kv)
    oracle.verify(model, kvb, np.array([[root, g[0], g[1]]], np.int32), None, np.array([3], np.int32))
    oracle.kv_commit(kvb, np.array([2], np.int32), None)
    assert kva.seq_len[0] == kvb.seq_len[0] == kv.seq_len[0] + 3
    n = int(kva.seq_len[0])
    assert np.array_equal(kva.k_bits[:, :, :, :n], kvb.k_bits[:, :, :, :n])
    assert np.array_equal(kva.v_bits[:, :, :, :n], kvb.v_bits[:, :, :, :n])
    nxt = np.array([[g[2]]], np.int32)
    ra = oracle.verify(model, kva, nxt, None, np.array([1], np.int32))
    rb = oracle.verify(model, kvb, nxt, None, np.array([1], np.int32))
    assert np.array_equal(ra.logits, rb.logits)


def test_int8_model_tracks_bf16_model(setup):
    """Sanity only (Section 4.5: quantisation should rarely flip the top-1): logits of the int8-weight
    model stay close to those of the bf16-weight model built from the same masters."""
    shape, model, kv, root = setup
    mb = oracle_model(shape, seed=0, int8=False)
    blk = np.array([[root, 1, 2, 3, 4]], np.int32)
    ra = oracle.verify(model, _copy(kv), blk, None, np.array([5], np.int32))
    rb = oracle.verify(mb, _copy(kv), blk, None, np.array([5], np.int32))
    assert np.max(np.abs(ra.logits - rb.logits)) < 0.1 * np.max(np.abs(rb.logits))
