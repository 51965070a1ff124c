"""The W8A8 kernels against the oracle, through the C ABI (needs a GPU): smoothing factors, smoothed weight
quantisation, fused activation smoothing + quantisation, integer GEMM with dequantisation
(Section 3.2 Eq. 4-8, Section 3.3 Eq. 9-10).  Integer codes and int32 accumulators: bit for bit."""
import numpy as np
import pytest
import torch

from oracle import quasar_oracle as qo
from paper_2603_01399_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _bits(t):
    return synth.bf16_bits(t)


def _f32(t):
    return qo.bf16_bits_to_f32(_bits(t))


@pytest.mark.parametrize("n,k,alpha", [(48, 64, 0.5), (1376, 688, 0.5), (512, 4096, 0.75), (64, 256, 0.0), (64, 256, 1.0)])
def test_smoothing_factors_and_smoothed_weights_bit_exact(n, k, alpha):
    w = synth.normal_bf16((n, k), 0.02, seed=n + k, device="cuda")
    a = torch.empty(k, dtype=torch.float32, device="cuda").uniform_(0.5, 40.0, generator=torch.Generator("cuda").manual_seed(k))
    a[3] = 0.0                                           # a dead channel: s = 1
    w[:, 5] = 0                                          # a zero weight column: s = 1
    s = binding.quasar_smoothing_factors(a, w, alpha)
    os_ = qo.smoothing_factors(a.cpu().numpy(), _f32(w), alpha)
    assert np.array_equal(s.cpu().numpy().view(np.uint32), os_.view(np.uint32))
    assert s[3] == 1.0 and s[5] == 1.0
    q, d = binding.quasar_quantize_weights_smoothed(w, s)
    oq, od = qo.quantize(qo.smooth_weights(_f32(w), os_))
    assert np.array_equal(d.cpu().numpy().view(np.uint32), od.view(np.uint32))
    assert np.array_equal(q.cpu().numpy(), oq)
    # without factors it is quasar_quantize
    q0, d0 = binding.quasar_quantize_weights_smoothed(w, None)
    q1, d1 = binding.quasar_quantize(w)
    assert torch.equal(q0, q1) and torch.equal(d0, d1)


@pytest.mark.parametrize("m,k", [(1, 16), (5, 688), (6, 4096), (17, 12288), (72, 4096)])
def test_activation_quantisation_bit_exact(m, k):
    x = synth.normal_bf16((m, k), 1.0, seed=m * 7 + k, device="cuda")
    x[0, :] = 0                                          # an all-zero token: delta 1, codes 0
    if m > 1:
        x[1, 7 % k] = 300.0                              # an outlier
    s = torch.empty(k, dtype=torch.float32, device="cuda").uniform_(0.05, 3.0, generator=torch.Generator("cuda").manual_seed(m))
    for sv in (s, None):
        q, d = binding.quasar_quantize_activations(x, sv)
        oq, od = qo.quantize_activations(_f32(x).astype(np.float64), None if sv is None else sv.cpu().numpy())
        assert np.array_equal(d.cpu().numpy().view(np.uint32), od.view(np.uint32))
        assert np.array_equal(q.cpu().numpy(), oq)


def _case(m, n, k, seed, smooth=True):
    w = synth.normal_bf16((n, k), 0.02, seed=seed, device="cuda")
    x = synth.normal_bf16((m, k), 1.0, seed=seed + 1, device="cuda")
    s = None
    if smooth:
        a = torch.empty(k, dtype=torch.float32, device="cuda").uniform_(0.5, 30.0, generator=torch.Generator("cuda").manual_seed(seed))
        s = binding.quasar_smoothing_factors(a, w, 0.5)
    wq, dw = binding.quasar_quantize_weights_smoothed(w, s)
    return x, s, wq, dw


@pytest.mark.parametrize("m,n,k", [(8, 64, 64), (1, 16, 16), (5, 1376, 688), (17, 512, 256), (6, 100, 4096), (72, 200, 1040),
                                   (80, 64, 2048)])
def test_linear_w8a8_accumulators_bit_exact_and_output_close(m, n, k):
    x, s, wq, dw = _case(m, n, k, seed=m * 31 + n + k)
    y, acc = binding.quasar_linear_w8a8(x, s, wq, dw, out_f32=True, want_acc=True)
    sn = None if s is None else s.cpu().numpy()
    xq, dx = qo.quantize_activations(_f32(x).astype(np.float64), sn)
    want_acc = qo.int_matmul(xq, wq.cpu().numpy())
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), want_acc)
    want = qo.linear_w8a8(_f32(x).astype(np.float64), sn, wq.cpu().numpy(), dw.cpu().numpy())
    got = y.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - want) <= 2e-7 * np.abs(want) + 1e-30)            # two fp32 roundings
    # bf16 output with a residual: rounded where the decoder layer rounds
    res = synth.normal_bf16((m, n), 1.0, seed=9, device="cuda")
    yb = binding.quasar_linear_w8a8(x, s, wq, dw, residual=res)
    ref = qo.bf16_round(qo.bf16_round(want) + _f32(res).astype(np.float64))
    gb = yb.float().cpu().numpy().astype(np.float64)
    assert np.mean(gb != ref) < 2e-3 and np.all(np.abs(gb - ref) <= 2.0 ** -7 * np.maximum(np.abs(ref), 1e-3))


def test_linear_w8a8_qwen3_8b_shapes_sampled():
    """The five matrix shapes of the benchmark at 6 and 40 rows: accumulators of sampled output channels
    against the oracle's exact integer product."""
    rng = np.random.default_rng(0)
    for k, n in [(4096, 6144), (4096, 4096), (4096, 24576), (12288, 4096), (4096, 151936)]:
        for m in (6, 40):
            x, s, wq, dw = _case(m, n, k, seed=k + n + m)
            y, acc = binding.quasar_linear_w8a8(x, s, wq, dw, out_f32=True, want_acc=True)
            cols = np.unique(np.concatenate([rng.integers(0, n, 64), [0, n - 1, n // 2]]))
            xq, dx = qo.quantize_activations(_f32(x).astype(np.float64), s.cpu().numpy())
            wsub = wq[torch.from_numpy(cols).cuda()].cpu().numpy()
            want_acc = qo.int_matmul(xq, wsub)
            assert np.array_equal(acc[:, torch.from_numpy(cols).cuda()].cpu().numpy().astype(np.int64), want_acc)
            want = want_acc.astype(np.float64) * (dw.cpu().numpy()[cols].astype(np.float64)[None, :] * dx.astype(np.float64)[:, None])
            got = y[:, torch.from_numpy(cols).cuda()].cpu().numpy().astype(np.float64)
            assert np.all(np.abs(got - want) <= 2e-7 * np.abs(want) + 1e-30)


# ---- the whole pass with the W8A8 verifier, tiny models, against the W8A8 oracle ---------------------
import oracle                                                                     # noqa: E402
from tests.common import (FULLWIDTH_MEAN_TOL, FULLWIDTH_SHARE, FULLWIDTH_WORST_TOL, fullwidth_stats, gpu_model,   # noqa: E402
                          margins, oracle_greedy_continuation, oracle_model, prefill_oracle)

S_MAX = 128


@pytest.fixture(scope="module", params=["tiny", "tiny_qknorm"])
def world(request):
    shape = synth.SHAPES[request.param]
    om = oracle_model(shape, seed=0, int8=True, act_int8=True)
    gm = gpu_model(shape, seed=0, int8=True, max_seq=S_MAX, act_int8=True)
    # offline preparation on the GPU == the oracle's, bit for bit (factors, codes, step sizes)
    for l in range(shape.n_layers):
        for nm, ol in (("qkv", om.layers[l].qkv), ("o", om.layers[l].o), ("gateup", om.layers[l].gateup),
                       ("down", om.layers[l].down)):
            assert np.array_equal(gm.tensors[f"l{l}.{nm}_smooth"].cpu().numpy().view(np.uint32), ol.smooth.view(np.uint32))
            assert np.array_equal(gm.tensors[f"l{l}.{nm}_w"].cpu().numpy(), ol.w)
            assert np.array_equal(gm.tensors[f"l{l}.{nm}_delta"].cpu().numpy(), ol.delta)
    assert np.array_equal(gm.tensors["lm_w"].cpu().numpy(), om.lm_head.w)
    okv = oracle.new_kv(om, 1, S_MAX)
    toks = synth.uniform_tokens((64,), shape.vocab, synth.sub_seed(2, "tokens"))
    prefill_oracle(om, okv, toks[:63].numpy(), chunk=8)
    return shape, om, gm, okv, int(toks[63])


def _run(shape, gm, okv, tokens, parents, bl, path=0, trace=False):
    B, T = tokens.shape
    k = torch.from_numpy(okv.k_bits.view(np.int16).copy()).view(torch.bfloat16).cuda()
    v = torch.from_numpy(okv.v_bits.view(np.int16).copy()).view(torch.bfloat16).cuda()
    kv = binding.KVCache(shape, okv.seq_len.shape[0], okv.s_max, k=k, v=v, seq_len=torch.from_numpy(okv.seq_len.copy()).cuda())
    buf = binding.VerifyBuffers(gm, B, T, tree=parents is not None)
    buf.tokens.copy_(torch.from_numpy(tokens))
    buf.block_len.copy_(torch.from_numpy(bl))
    if parents is not None:
        buf.parents.copy_(torch.from_numpy(parents))
    tr = torch.zeros(gm.trace_bytes(B, T), dtype=torch.uint8, device="cuda") if trace else None
    gm.set_path(path)
    gm.set_trace(tr)
    try:
        binding.quasar_verify(gm, kv, buf)
        torch.cuda.synchronize()
    finally:
        gm.set_trace(None)
        gm.set_path(0)
    assert int(buf.status[0]) == 0
    return kv, buf, (binding.split_trace(gm, tr, B, T) if trace else None)


# End to end, the element test of the weight-only pass cannot be asked of W8A8: where the two sides differ by
# one bf16 rounding in an activation (fp32 against fp64 in a norm or in the attention), the element's int8
# code moves with probability ~ |x| 2^-8 / delta_x, and one code step is 1/127 of the row's maximum - the
# method turns a rounding into a quantisation step.  So: (1) every W8A8 linear layer of the pass is checked
# on its own from the input the GPU itself recorded (within one bf16 rounding: the integer product is exact);
# (2) end to end the criterion of the full-width tests (share of the logits inside the element test, bounded
# mean and worst difference) and exact top-1 / acceptance on margin-safe rows.
def _check(r, buf, bl):
    lg = buf.logits.cpu().numpy()
    for b in range(len(bl)):
        T = int(bl[b])
        inside, mean, worst = fullwidth_stats(lg[b, :T], r.logits[b, :T])
        assert inside >= FULLWIDTH_SHARE and mean <= FULLWIDTH_MEAN_TOL and worst <= FULLWIDTH_WORST_TOL, (inside, mean, worst)
        safe = margins(r.logits[b, :T]) > max(5e-2, 2 * worst)
        assert np.array_equal(lg[b, :T].argmax(-1)[safe], r.top1[b, :T][safe])
        path = [int(p) for p in r.accept_path[b] if p >= 0]
        if all(safe[p] for p in path):
            assert int(buf.accept_len[b]) == int(r.accept_len[b]) and int(buf.bonus[b]) == int(r.bonus[b])


def _np(t):
    return t.float().cpu().numpy().astype(np.float64)


def _one_rounding(name, got, want, prev=None):
    mag = np.abs(want) if prev is None else np.abs(want) + np.abs(prev) + np.abs(want - prev)
    tol = 2.5 * 2.0 ** -8 * np.maximum(mag, np.sqrt(np.mean(mag ** 2))) + 1e-6
    assert np.all(np.abs(got - want) <= tol), f"{name}: worst {np.abs(got - want).max():.3e}"
    assert np.mean(got != want) < 0.02, f"{name}: {np.mean(got != want):.4f} of the elements differ"


def _teacher_forced_linears(shape, om, tr, T, logits_gpu):
    """Each W8A8 linear layer recomputed by the oracle from the tensor the GPU recorded as its input."""
    R = qo.bf16_round
    for l in range(shape.n_layers):
        ly = om.layers[l]
        h1 = _np(tr[f"l{l}.h1"][0, :T])
        _one_rounding(f"l{l}.qkv", _np(tr[f"l{l}.qkv"][0, :T]), R(ly.qkv(h1)))
        attn = _np(tr[f"l{l}.attn"][0, :T])
        x_in = _np(tr["embed"][0, :T]) if l == 0 else _np(tr[f"l{l - 1}.x_mlp"][0, :T])
        x_attn = _np(tr[f"l{l}.x_attn"][0, :T])
        _one_rounding(f"l{l}.x_attn", x_attn, R(x_in + R(ly.o(attn))), prev=x_in)
        act = _np(tr[f"l{l}.act"][0, :T])
        _one_rounding(f"l{l}.x_mlp", _np(tr[f"l{l}.x_mlp"][0, :T]), R(x_attn + R(ly.down(act))), prev=x_attn)
    hf = _np(tr["hf"][0, :T])
    want = om.lm_head(hf)
    assert np.all(np.abs(logits_gpu[0, :T] - want) <= 2e-6 * np.maximum(np.abs(want), 1.0))


@pytest.mark.parametrize("path", [1, 0])
def test_w8a8_pass_chain_and_tree_against_the_w8a8_oracle(world, path):
    shape, om, gm, okv, root = world
    copy = lambda kv: oracle.KVCache(kv.k_bits.copy(), kv.v_bits.copy(), kv.seq_len.copy())
    g = oracle_greedy_continuation(om, okv, root, 5)
    # chain: the model's own continuation with one wrong token in the middle
    tokens = np.array([[root, g[0], g[1], (g[2] + 1) % shape.vocab, g[3]]], np.int32)
    bl = np.array([5], np.int32)
    r = oracle.verify(om, copy(okv), tokens, None, bl)
    assert int(r.accept_len[0]) == 2
    _, buf, _ = _run(shape, gm, okv, tokens, None, bl, path)
    _check(r, buf, bl)
    # tree of eight rows with the greedy path on one branch
    parents = np.array([[-1, 0, 0, 1, 2, 2, 4, 5]], np.int32)
    tokens = np.array([[root, 7, g[0], 9, g[1], 11, g[2], 13]], np.int32)
    bl = np.array([8], np.int32)
    r = oracle.verify(om, copy(okv), tokens, parents, bl)
    assert int(r.accept_len[0]) == 3
    _, buf, _ = _run(shape, gm, okv, tokens, parents, bl, path)
    _check(r, buf, bl)
    if margins(r.logits[0]).min() > 0.1:
        assert np.array_equal(buf.accept_path[0].cpu().numpy(), r.accept_path[0])
    if path == 1:
        _, buf, tr = _run(shape, gm, okv, tokens, parents, bl, path, trace=True)
        _teacher_forced_linears(shape, om, tr, 8, buf.logits.cpu().numpy().astype(np.float64))
