"""Pins of the oracle's W8A8 linear layer (Section 3.2 Eq. 4-8, Section 3.3 Eq. 9-10): smoothing factors,
smoothed weights, per-token activation quantisation, exact integer accumulation, dequantisation (CPU only)."""
import os

import numpy as np
import pytest

import oracle
from oracle import quasar_oracle as qo
from paper_2603_01399_b200 import synth
from tests.common import oracle_greedy_continuation, prefill_oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _bf16(a):
    return qo.bf16_round(np.asarray(a, np.float64))


def test_smoothing_identity_eq4():
    """Y = W X = (W diag(s)^-1)(diag(s) X) for any positive s."""
    rng = np.random.default_rng(0)
    w = rng.normal(size=(24, 40))
    x = rng.normal(size=(5, 40))
    s = rng.uniform(0.1, 9.0, 40)
    y = x @ w.T
    y2 = (x * s[None, :]) @ (w / s[None, :]).T
    assert np.max(np.abs(y - y2)) <= 1e-12 * np.max(np.abs(y))


def test_smoothing_factors_closed_forms_eq5():
    w = np.array([[1.0, -0.5, 0.0, 2.0], [-0.25, 0.125, 0.0, -8.0]], np.float32)       # column maxima 1, .5, 0, 8
    a = np.array([4.0, 2.0, 3.0, 0.0], np.float32)
    s = qo.smoothing_factors(a, w, 0.5)
    assert s.dtype == np.float32
    assert list(s) == [0.5, 0.5, 1.0, 1.0]          # sqrt(1/4), sqrt(.5/2); a zero maximum on either side -> 1
    assert list(qo.smoothing_factors(a, w, 1.0)[:2]) == [0.25, 0.5]                    # alpha = 1: 1 / max|X_j|
    assert list(qo.smoothing_factors(a, w, 0.0)[:2]) == [1.0, 0.5]                     # alpha = 0: max|W_j|
    # after smoothing with alpha = 1/2 the two sides have the same maximum per channel: sqrt(max|X_j| max|W_j|)
    rng = np.random.default_rng(1)
    w = rng.normal(size=(16, 32)).astype(np.float32)
    a = rng.uniform(0.5, 30.0, 32).astype(np.float32)
    s = qo.smoothing_factors(a, w, 0.5).astype(np.float64)
    wmax = np.abs(w).max(0)
    assert np.allclose(a * s, wmax / s, rtol=1e-6)
    assert np.allclose(np.abs(qo.smooth_weights(w, s.astype(np.float32))).max(0), np.sqrt(a * wmax), rtol=1e-6)


def test_activation_quantisation_is_the_same_operator_as_for_weights():
    """Q(., delta) of Eq. 6-7 and Eq. 9 is one operator: the hand-worked rows hold for activations too."""
    for line in open(os.path.join(GOLD, "quantize_hand_cases.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        ws, ds, qs = [p.strip() for p in line.split("|")]
        x = np.array([[float(v) for v in ws.split()]], np.float64)
        num, den = ds.split("/")
        q, dx = qo.quantize_activations(x, None)
        assert dx[0] == np.float32(np.float32(num) / np.float32(den))
        assert list(q[0]) == [int(v) for v in qs.split()]
    # with smoothing the operator sees x * s: row [1, 2] with s = [4, 0.5] is the row [4, 1]
    q, dx = qo.quantize_activations(np.array([[1.0, 2.0]]), np.array([4.0, 0.5], np.float32))
    assert dx[0] == np.float32(4.0) / np.float32(127.0) and list(q[0]) == [127, 32]    # 1 / (4/127) = 31.75 -> 32
    # error bound |x~ - q delta| <= delta / 2 per element
    rng = np.random.default_rng(2)
    x = _bf16(rng.normal(size=(7, 96)) * 3)
    s = rng.uniform(0.2, 5.0, 96).astype(np.float32)
    q, dx = qo.quantize_activations(x, s)
    xt = (x.astype(np.float32) * s).astype(np.float64)
    err = np.abs(xt - q.astype(np.float64) * dx.astype(np.float64)[:, None])
    assert np.all(err <= dx.astype(np.float64)[:, None] * (0.5 + 2.0 ** -22))
    assert np.all(np.abs(q).max(1) == 127)


def test_integer_accumulators_against_a_triple_loop():
    rng = np.random.default_rng(3)
    xq = rng.integers(-127, 128, (4, 37)).astype(np.int8)
    wq = rng.integers(-127, 128, (9, 37)).astype(np.int8)
    acc = qo.int_matmul(xq, wq)
    for m in range(4):
        for n in range(9):
            t = 0
            for k in range(37):
                t += int(xq[m, k]) * int(wq[n, k])
            assert int(acc[m, n]) == t
    # the largest contraction of the benchmark shapes stays inside int32 even at full scale
    assert 17408 * 127 * 127 < 2 ** 31


def test_w8a8_linear_is_exact_when_both_operands_sit_on_their_grids():
    """x = 2^-3 * integers with row maximum 127 and weights = 2^-5 * integers with row maximum 127 are
    reproduced exactly by Q, so Eq. 10 returns W x exactly."""
    rng = np.random.default_rng(4)
    xi = rng.integers(-127, 128, (3, 64)); xi[:, 0] = 127
    wi = rng.integers(-127, 128, (6, 64)); wi[:, 1] = -127
    x = xi * 2.0 ** -3
    w = (wi * 2.0 ** -5).astype(np.float32)
    wq, dw = qo.quantize(w)
    assert np.array_equal(wq, wi) and np.all(dw == np.float32(2.0 ** -5))
    y = qo.linear_w8a8(x, None, wq, dw)
    assert np.array_equal(y, x @ w.astype(np.float64).T)


def test_w8a8_error_bound_and_what_smoothing_buys():
    """|Y - W X| is bounded by the two rounding errors; with an outlier activation channel the smoothed
    layer (alpha = 1/2) is several times closer to W X than the unsmoothed one."""
    rng = np.random.default_rng(5)
    K, N, M = 256, 48, 6
    w = _bf16(rng.normal(size=(N, K)) * 0.02).astype(np.float32)
    x = _bf16(rng.normal(size=(M, K)))
    x[:, 7] = _bf16(x[:, 7] * 60.0)                       # a systematic outlier channel
    exact = x @ w.astype(np.float64).T
    a = np.abs(x).max(0).astype(np.float32)              # calibrated on the data itself
    errs = {}
    for name, s in (("plain", None), ("smoothed", qo.smoothing_factors(a, w, 0.5))):
        wt = w if s is None else qo.smooth_weights(w, s)
        wq, dw = qo.quantize(wt)
        y = qo.linear_w8a8(x, s, wq, dw)
        xq, dx = qo.quantize_activations(x, s)
        # |w~ x~ - (q_w dw)(q_x dx)| <= |w~| dx/2 + |x~| dw/2 + dw dx / 4 per term
        xt = np.abs(x if s is None else x * s.astype(np.float64)[None, :])
        wa = np.abs(wt.astype(np.float64))
        bound = (xt @ (np.ones_like(wa) * dw.astype(np.float64)[:, None]).T) * 0.5 \
            + (np.ones_like(xt) * dx.astype(np.float64)[:, None]) @ wa.T * 0.5 \
            + K * dw.astype(np.float64)[None, :] * dx.astype(np.float64)[:, None] * 0.25
        assert np.all(np.abs(y - exact) <= bound * (1 + 1e-5) + 1e-12), name
        errs[name] = float(np.sqrt(np.mean((y - exact) ** 2)))
    assert errs["smoothed"] < errs["plain"] / 3, errs


def test_no_smoothing_is_plain_w8a8_on_the_unsmoothed_weights():
    rng = np.random.default_rng(6)
    w = _bf16(rng.normal(size=(10, 32)) * 0.02).astype(np.float32)
    x = _bf16(rng.normal(size=(3, 32)))
    ones = np.ones(32, np.float32)
    wq, dw = qo.quantize(w)
    wq1, dw1 = qo.quantize(qo.smooth_weights(w, ones))
    assert np.array_equal(wq, wq1) and np.array_equal(dw, dw1)
    assert np.array_equal(qo.linear_w8a8(x, ones, wq, dw), qo.linear_w8a8(x, None, wq, dw))


# ---- the whole pass with the W8A8 verifier ----------------------------------------------------------
@pytest.fixture(scope="module", params=["tiny", "tiny_qknorm"])
def setup(request):
    shape = synth.SHAPES[request.param]
    get = lambda kind, layer=0: (synth.embedding(shape, 0) if kind == "embed" else
                                 synth.gain(shape, kind, layer, 0) if "norm" in kind else
                                 synth.matrix(shape, kind, layer, 0))
    model = oracle.build_model(shape, lambda kind, layer: synth.bf16_bits(get(kind, layer)), int8=True, act_int8=True,
                               get_act_absmax=lambda kind, layer: synth.activation_absmax(shape, kind, layer, 0).numpy())
    kv = oracle.new_kv(model, 1, 96)
    toks = synth.uniform_tokens((64,), shape.vocab, synth.sub_seed(2, "tokens"))
    prefill_oracle(model, kv, toks[:63].numpy(), chunk=8)
    return shape, model, kv, int(toks[63])


def _copy(kv):
    return oracle.KVCache(kv.k_bits.copy(), kv.v_bits.copy(), kv.seq_len.copy())


def test_w8a8_pass_block_equals_row_by_row_and_own_draft_is_accepted(setup):
    """Activations are quantised per token, so the rows of a block stay independent: one call over the block
    equals decode steps with commits, bit for bit; and the model's own greedy continuation is accepted."""
    shape, model, kv, root = setup
    assert model.layers[0].qkv.act_int8 and model.layers[0].qkv.smooth is not None
    g = oracle_greedy_continuation(model, kv, root, 5)
    tokens = np.array([[root] + g[:4]], np.int32)
    r = oracle.verify(model, _copy(kv), tokens, None, np.array([5], np.int32))
    assert r.accept_len[0] == 4 and r.bonus[0] == g[4]
    kv2 = _copy(kv)
    for i in range(5):
        one = oracle.verify(model, kv2, tokens[:, i:i + 1].copy(), None, np.array([1], np.int32))
        assert np.array_equal(one.logits[0, 0], r.logits[0, i])
        oracle.kv_commit(kv2, np.array([0], np.int32), None)
    # a chain written as a tree gives the same logits
    par = np.array([[-1, 0, 1, 2, 3]], np.int32)
    rt = oracle.verify(model, _copy(kv), tokens, par, np.array([5], np.int32))
    assert np.array_equal(rt.logits, r.logits)


def test_w8a8_model_stays_close_to_the_weight_only_model(setup):
    """Quantising the activations as well moves the logits by a few per cent of their spread, no more
    (the paper's premise that W8A8 preserves the distribution, Section 4.5, on random weights)."""
    shape, model, kv, root = setup
    get = lambda kind, layer=0: (synth.embedding(shape, 0) if kind == "embed" else
                                 synth.gain(shape, kind, layer, 0) if "norm" in kind else
                                 synth.matrix(shape, kind, layer, 0))
    w8a16 = oracle.build_model(shape, lambda kind, layer: synth.bf16_bits(get(kind, layer)), int8=True)
    tokens = np.array([[root, 5, 6, 7]], np.int32)
    bl = np.array([4], np.int32)
    a = oracle.verify(model, _copy(kv), tokens, None, bl).logits
    b = oracle.verify(w8a16, _copy(kv), tokens, None, bl).logits
    assert np.abs(a - b).mean() < 0.1 * b.std()
