"""Pins for the oracle's single steps (CPU only).  Each test checks the oracle against
something other than itself: hand-worked values, closed forms, brute force, or a library
routine that the oracle does not call."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import quasar_oracle as qo

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- bf16 rounding
def test_bf16_round_matches_torch_cast():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(200000) * 10.0 ** rng.integers(-35, 35, 200000)).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy().astype(np.float64)
    got = qo.bf16_round(x.astype(np.float64))
    assert np.array_equal(want, got)


def test_bf16_round_hand_cases():
    # 8 significant bits: 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even mantissa (1.0)
    assert qo.bf16_round(1 + 2.0 ** -8) == 1.0
    assert qo.bf16_round(1 + 3 * 2.0 ** -8) == 1 + 2.0 ** -6
    # a value just above the tie must round up even though fp32 would first round it onto the tie
    assert qo.bf16_round(1 + 2.0 ** -8 + 2.0 ** -40) == 1 + 2.0 ** -7
    assert qo.bf16_round(-0.0) == 0.0 and qo.bf16_round(0.0) == 0.0
    assert qo.bf16_round(255.5) == 256.0 and qo.bf16_round(254.5) == 254.0


def test_bf16_bits_roundtrip_all_patterns():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    v = qo.bf16_bits_to_f64(bits)
    finite = np.isfinite(v)
    back = qo.f64_to_bf16_bits(v[finite])
    want = bits[finite]
    # -0.0 and +0.0 keep their sign bit through float32
    assert np.array_equal(back, want)


# ---------------------------------------------------------------- quantise (Eq. 6-7)
def _hand_cases():
    out = []
    with open(os.path.join(GOLD, "quantize_hand_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w, d, q = [s.strip() for s in line.split("|")]
            a, b = d.split("/")
            out.append((np.array([float(t) for t in w.split()], np.float32),
                        np.float32(float(a)) / np.float32(float(b)),
                        np.array([int(t) for t in q.split()], np.int8)))
    return out


def test_quantize_hand_cases():
    for w, delta, q in _hand_cases():
        gq, gd = qo.quantize(w[None, :])
        assert gd[0] == delta and gd.dtype == np.float32
        assert np.array_equal(gq[0], q), (w, gq, q)


def test_quantize_error_bound_and_range():
    rng = np.random.default_rng(1)
    w = torch.from_numpy((rng.standard_normal((64, 512)) * 0.02).astype(np.float32)).to(torch.bfloat16).float().numpy()
    q, d = qo.quantize(w)
    assert q.dtype == np.int8 and q.min() >= -127
    assert np.all(np.max(np.abs(q.astype(np.int32)), axis=1) == 127)
    err = np.abs(w.astype(np.float64) - qo.dequantize(q, d))
    # w/delta is an fp32 quotient of magnitude <= 127, so it carries up to 127 * 2^-24 of rounding
    # error before the half-to-even step: the bound is half a step plus that much
    bound = d.astype(np.float64)[:, None] * (0.5 + 127 * 2.0 ** -23)
    assert np.all(err <= bound)


def test_quantize_idempotent_on_own_grid():
    rng = np.random.default_rng(2)
    q0 = rng.integers(-127, 128, (16, 64)).astype(np.int8)
    q0[:, 0] = 127                                   # absmax attained
    for delta in (1.0, 0.5, 2.0 ** -9):               # power-of-two steps: q*delta exact in fp32
        w = (q0.astype(np.float32) * np.float32(delta))
        q, d = qo.quantize(w)
        assert np.array_equal(q, q0)
        assert np.all(d == np.float32(127 * delta) / np.float32(127))


def test_quantize_every_bf16_value_against_fp64_restatement():
    """All finite bf16 magnitudes as one long row per scale; away from rounding ties the fp32
    computation must agree with exact rational arithmetic done in fp64."""
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    vals = qo.bf16_bits_to_f64(bits)
    for amax in (1.0, 0.0712890625, 3.0):             # bf16-representable maxima
        v = vals[np.isfinite(vals) & (np.abs(vals) <= amax)]
        row = np.concatenate([[amax], v]).astype(np.float32)
        q, d = qo.quantize(row[None, :])
        exact = row.astype(np.float64) * 127.0 / amax
        frac = np.abs(exact - np.floor(exact) - 0.5)
        safe = frac > 1e-4                            # away from .5 ties
        assert np.array_equal(q[0][safe], np.clip(np.rint(exact[safe]), -127, 127).astype(np.int8))
        assert np.all(np.abs(q[0].astype(np.float64) - exact) <= 0.5 + 1e-4)


def test_quantize_zero_and_constant_rows():
    q, d = qo.quantize(np.zeros((2, 8), np.float32))
    assert np.all(q == 0) and np.all(d == 1.0)
    q, d = qo.quantize(np.full((1, 8), -0.375, np.float32))
    assert np.all(q == -127) and d[0] == np.float32(0.375) / np.float32(127)


# ---------------------------------------------------------------- quantised linear (Eq. 8 / 10)
def test_linear_brute_force_triple_loop():
    rng = np.random.default_rng(3)
    M, K, N = 5, 48, 24
    x = qo.bf16_round(rng.standard_normal((M, K)))
    q = rng.integers(-127, 128, (N, K)).astype(np.int8)
    d = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    got = qo.linear(x, q, d)
    for m in range(M):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                acc += float(x[m, k]) * int(q[n, k])
            assert got[m, n] == pytest.approx(acc * float(d[n]), rel=1e-13, abs=1e-300)


def test_linear_exact_integer_case_and_scaling():
    rng = np.random.default_rng(4)
    x = rng.integers(-8, 9, (3, 64)).astype(np.float64)
    q = rng.integers(-127, 128, (10, 64)).astype(np.int8)
    ones = np.ones(10, np.float32)
    got = qo.linear(x, q, ones)
    want = x.astype(np.int64) @ q.astype(np.int64).T
    assert np.array_equal(got, want.astype(np.float64))
    assert np.array_equal(qo.linear(2 * x, q, ones), 2 * got)
    # transposed operand or wrong scale axis would break this: scale row n only
    d = np.arange(1, 11).astype(np.float32)
    assert np.array_equal(qo.linear(x, q, d), want * d[None, :].astype(np.float64))


def test_linear_concatenation_property():
    rng = np.random.default_rng(5)
    x = qo.bf16_round(rng.standard_normal((4, 32)))
    qs = [rng.integers(-127, 128, (n, 32)).astype(np.int8) for n in (8, 4, 4)]
    ds = [rng.uniform(1e-3, 1e-2, q.shape[0]).astype(np.float32) for q in qs]
    fused = qo.linear(x, np.concatenate(qs), np.concatenate(ds))
    parts = np.concatenate([qo.linear(x, q, d) for q, d in zip(qs, ds)], axis=1)
    assert np.array_equal(fused, parts)


def test_linear_bf16_weight_sibling_matches_torch_double():
    rng = np.random.default_rng(6)
    w = torch.from_numpy(rng.standard_normal((12, 40)).astype(np.float32)).to(torch.bfloat16)
    x = torch.from_numpy(rng.standard_normal((3, 40)).astype(np.float32)).to(torch.bfloat16)
    lin = qo.Linear(w.view(torch.int16).numpy().view(np.uint16), None)
    got = lin(x.double().numpy())
    want = (x.double() @ w.double().T).numpy()
    assert np.allclose(got, want, rtol=1e-14, atol=0)


# ---------------------------------------------------------------- RMSNorm / SiLU / RoPE
def test_rmsnorm_closed_forms():
    g = np.array([0.5, 2.0, -1.0, 3.0])
    y = qo.rmsnorm(np.full((1, 4), -7.0), g, 0.0)
    assert np.allclose(y, -g)                        # constant vector -> sign * gain
    x = np.array([[3.0, 4.0, 0.0, 0.0]])            # mean square = 25/4
    assert np.allclose(qo.rmsnorm(x, np.ones(4), 0.0), x / 2.5)
    # eps enters under the root, added to the mean square
    assert np.allclose(qo.rmsnorm(x, np.ones(4), 0.75), x / math.sqrt(7.0))
    want = torch.nn.functional.rms_norm(torch.tensor(x), (4,), torch.tensor(g), 1e-6).numpy()
    assert np.allclose(qo.rmsnorm(x, g, 1e-6), want, rtol=1e-14)


def test_silu_closed_forms():
    assert qo.silu(np.array(0.0)) == 0.0
    assert qo.silu(np.array(1.0)) == pytest.approx(1 / (1 + math.exp(-1)))
    x = np.linspace(-5, 5, 11)
    assert np.allclose(qo.silu(x) - qo.silu(-x), x)  # silu(x) - silu(-x) = x
    assert np.allclose(qo.silu(x), torch.nn.functional.silu(torch.tensor(x)).numpy(), rtol=1e-14)


def test_rope_properties():
    rng = np.random.default_rng(7)
    D = 16
    x = rng.standard_normal((5, D))
    assert np.array_equal(qo.rope(x, np.zeros(5), 1e6), x)        # position 0 is the identity
    y = qo.rope(x, np.arange(5) * 37, 1e6)
    for i in range(D // 2):                                         # pair (i, i + D/2) keeps its norm
        assert np.allclose(x[:, i] ** 2 + x[:, i + D // 2] ** 2, y[:, i] ** 2 + y[:, i + D // 2] ** 2)
    q, k = rng.standard_normal(D), rng.standard_normal(D)
    a = qo.rope(q, np.array(11), 1e6) @ qo.rope(k, np.array(4), 1e6)
    b = qo.rope(q, np.array(1011), 1e6) @ qo.rope(k, np.array(1004), 1e6)
    assert a == pytest.approx(b, abs=1e-10)                         # depends on the offset only


def test_rope_explicit_angles():
    # D = 4, theta = 100: inv_freq = [1, 100^(-1/2)] = [1, 0.1]
    x = np.array([1.0, 2.0, 3.0, 4.0])
    p = 3.0
    y = qo.rope(x, np.array(p), 100.0)
    c0, s0, c1, s1 = math.cos(3.0), math.sin(3.0), math.cos(0.3), math.sin(0.3)
    want = [1 * c0 - 3 * s0, 2 * c1 - 4 * s1, 3 * c0 + 1 * s0, 4 * c1 + 2 * s1]
    assert np.allclose(y, want, rtol=1e-15)


# ---------------------------------------------------------------- attention
def _dense_attention(q, k, v, allowed):
    T, G, D = q.shape
    out = np.zeros_like(q)
    for i in range(T):
        for g in range(G):
            js = [j for j in range(k.shape[0]) if allowed[i][j]]
            s = [sum(q[i, g, d] * k[j, d] for d in range(D)) / math.sqrt(D) for j in js]
            mx = max(s)
            e = [math.exp(t - mx) for t in s]
            z = sum(e)
            for d in range(D):
                out[i, g, d] = sum(e[n] * v[j, d] for n, j in enumerate(js)) / z
    return out


def test_attention_vs_dense_brute_force_tree_mask():
    rng = np.random.default_rng(8)
    parents = [-1, 0, 0, 1, 2, 3]
    T, G, D, P = len(parents), 2, 8, 5
    q = rng.standard_normal((T, G, D)); k = rng.standard_normal((P + T, D)); v = rng.standard_normal((P + T, D))
    mask = qo.ancestor_mask(parents)
    # the mask written out by hand for this tree
    hand = np.array([[1, 0, 0, 0, 0, 0], [1, 1, 0, 0, 0, 0], [1, 0, 1, 0, 0, 0],
                     [1, 1, 0, 1, 0, 0], [1, 0, 1, 0, 1, 0], [1, 1, 0, 1, 0, 1]], bool)
    assert np.array_equal(mask, hand)
    allowed = np.concatenate([np.ones((T, P), bool), hand], axis=1)
    assert np.allclose(qo.attention(q, k, v, P, mask), _dense_attention(q, k, v, allowed), rtol=1e-12)


def test_attention_special_cases():
    rng = np.random.default_rng(9)
    D = 8
    q = rng.standard_normal((1, 3, D)); v = rng.standard_normal((1, D)); k = rng.standard_normal((1, D))
    out = qo.attention(q, k, v, 0, np.ones((1, 1), bool))            # single key -> v
    assert np.allclose(out, np.broadcast_to(v, (1, 3, D)))
    k = np.zeros((6, D)); v = rng.standard_normal((6, D))            # uniform scores -> mean of V
    out = qo.attention(rng.standard_normal((1, 2, D)), k, v, 5, np.ones((1, 1), bool))
    assert np.allclose(out, np.broadcast_to(v.mean(0), (1, 2, D)))
    # chain mask == torch causal sdpa on the suffix rows
    T, P = 4, 3
    q = rng.standard_normal((T, 1, D)); k = rng.standard_normal((P + T, D)); v = rng.standard_normal((P + T, D))
    mask = qo.ancestor_mask([-1, 0, 1, 2])
    got = qo.attention(q, k, v, P, mask)[:, 0]
    full = torch.ones(T, P + T, dtype=torch.bool).tril(diagonal=P)
    want = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(q[:, 0])[None], torch.tensor(k)[None], torch.tensor(v)[None], attn_mask=full[None])[0].numpy()
    assert np.allclose(got, want, rtol=1e-10, atol=1e-12)


# ---------------------------------------------------------------- acceptance (Eq. 2 at T = 0)
def test_accept_chain_all_match_patterns():
    for gamma in range(0, 9):
        T = gamma + 1
        parents = list(range(-1, T - 1))
        for pat in itertools.product([0, 1], repeat=gamma):
            top1 = [100 + i for i in range(T)]
            tokens = [7] + [top1[i - 1] if pat[i - 1] else 5 for i in range(1, T)]
            n, bonus, path = qo.accept_greedy(tokens, parents, top1)
            want = 0
            while want < gamma and pat[want]:
                want += 1
            assert n == want and bonus == top1[want] and path == list(range(want + 1))
            assert 0 <= n <= gamma


def test_accept_tree_lowest_index_child_and_branching():
    parents = [-1, 0, 0, 0, 1, 1, 2, 3]
    tokens = [9, 5, 6, 6, 7, 8, 7, 7]
    top1 = [6, 0, 7, 7, 0, 0, 1, 2]
    n, bonus, path = qo.accept_greedy(tokens, parents, top1)   # root->2 (first '6'), 2->6 ('7')
    assert (n, bonus, path) == (2, 1, [0, 2, 6])
    top1[0] = 4                                                 # nothing matches
    assert qo.accept_greedy(tokens, parents, top1) == (0, 4, [0])
    top1[0] = 5; top1[1] = 8
    assert qo.accept_greedy(tokens, parents, top1) == (2, 0, [0, 1, 5])
