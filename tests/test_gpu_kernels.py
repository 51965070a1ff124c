"""Parity of single kernels against the oracle, through the C ABI (needs a GPU)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import quasar_oracle as qo
from paper_2603_01399_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _bits(t):
    return synth.bf16_bits(t)


# ---------------------------------------------------------------- quantise: bit-exact
@pytest.mark.parametrize("n,k", [(7, 16), (64, 688), (1376, 256), (513, 4096), (16, 17408)])
def test_quantize_bit_exact_random(n, k):
    w = synth.normal_bf16((n, k), 0.02, seed=n * 131 + k, device="cuda")
    w[0, :] = 0                                         # an all-zero row
    if n > 2:
        w[1, :] = w[1, 0]                               # a constant row
    q, d = binding.quasar_quantize(w)
    oq, od = qo.quantize(qo.bf16_bits_to_f32(_bits(w)))
    assert np.array_equal(d.cpu().numpy().view(np.uint32), od.view(np.uint32))
    assert np.array_equal(q.cpu().numpy(), oq)


def test_quantize_bit_exact_all_bf16_patterns():
    bits = torch.arange(65536, dtype=torch.int32).to(torch.int16)
    vals = bits.view(torch.bfloat16)
    finite = torch.isfinite(vals.float())
    v = vals[finite]
    v = v[: (v.numel() // 8) * 8]
    rows = []
    for amax in (1.0, 0.0712890625, 3.0, 3.3e38):
        r = v.clone()
        r[r.float().abs() > amax] = 0
        r[0] = amax
        rows.append(r)
    w = torch.stack(rows).contiguous().cuda()
    q, d = binding.quasar_quantize(w)
    oq, od = qo.quantize(qo.bf16_bits_to_f32(_bits(w)))
    assert np.array_equal(d.cpu().numpy().view(np.uint32), od.view(np.uint32))
    assert np.array_equal(q.cpu().numpy(), oq)


def test_linear_calls_of_different_widths_share_one_workspace():
    """A decoder layer runs its GEMMs of different widths through one workspace, narrow ones first: a
    call's partial sums must not land where a wider call keeps its arrival counters."""
    shapes = [(6144, 4096), (4096, 4096), (24576, 4096), (4096, 12288), (151936, 4096), (24576, 4096)]
    m = 6
    size = max(binding.quasar_linear_workspace_bytes(m, n, k) for n, k in shapes)
    shared = torch.zeros(size, dtype=torch.uint8, device="cuda")
    for i, (n, k) in enumerate(shapes):
        x = synth.normal_bf16((m, k), 1.0, seed=10 + i, device="cuda")
        q, d = binding.quasar_quantize(synth.normal_bf16((n, k), 0.02, seed=20 + i, device="cuda"))
        alone = binding.quasar_linear(x, q, d, out_f32=True)          # a zero-filled workspace of its own
        assert torch.equal(binding.quasar_linear(x, q, d, workspace=shared, out_f32=True), alone)


@pytest.mark.parametrize("k,n", [(4096, 6144), (4096, 4096), (4096, 24576), (12288, 4096), (4096, 151936)])
def test_quantize_bit_exact_qwen3_8b_shapes(k, n):
    w = synth.normal_bf16((n, k), 0.02, seed=k + n, device="cuda")
    q, d = binding.quasar_quantize(w)
    step = max(1, n // 4096)                             # every row's delta, a strided sample of rows for q
    wb = _bits(w)
    oq, od = qo.quantize(qo.bf16_bits_to_f32(wb[::step]))
    assert np.array_equal(d.cpu().numpy()[::step].view(np.uint32), od.view(np.uint32))
    assert np.array_equal(q.cpu().numpy()[::step], oq)
    # every row's step size: delta = absmax / 127 in IEEE fp32 (numpy on the host)
    absmax = w.float().abs().amax(dim=1).cpu().numpy()
    assert np.array_equal(d.cpu().numpy(), (absmax / np.float32(127.0)).astype(np.float32))


# ---------------------------------------------------------------- quantised linear
def _linear_case(m, n, k, int8, residual, out_f32, seed):
    x = synth.normal_bf16((m, k), 1.0, seed=seed, device="cuda")
    wm = synth.normal_bf16((n, k), 0.02, seed=seed + 1, device="cuda")
    res = synth.normal_bf16((m, n), 1.0, seed=seed + 2, device="cuda") if residual else None
    xo = qo.bf16_bits_to_f64(_bits(x))
    if int8:
        q, d = binding.quasar_quantize(wm)
        oq, od = qo.quantize(qo.bf16_bits_to_f32(_bits(wm)))
        assert np.array_equal(q.cpu().numpy(), oq)
        want = qo.linear(xo, oq, od)
        absw = qo.linear(np.abs(xo), np.abs(oq.astype(np.int16)).astype(np.float64), od)
        y = binding.quasar_linear(x, q, d, residual=res, out_f32=out_f32)
    else:
        wf = qo.bf16_bits_to_f64(_bits(wm))
        want = qo.linear(xo, wf, None)
        absw = qo.linear(np.abs(xo), np.abs(wf), None)
        y = binding.quasar_linear(x, wm, None, residual=res, out_f32=out_f32)
    torch.cuda.synchronize()
    acc_err = 4e-6 * absw + 1e-30                         # fp32 accumulation of K terms vs fp64
    if residual:
        r = qo.bf16_bits_to_f64(_bits(res))
        want2 = r + qo.bf16_round(want)
        got = y.float().cpu().numpy().astype(np.float64)
        tol = acc_err + 2.0 ** -7 * np.abs(want) + (0 if out_f32 else 2.0 ** -7 * np.abs(want2))
        assert np.all(np.abs(got - want2) <= tol)
    elif out_f32:
        got = y.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - want) <= acc_err + 1e-6 * np.abs(want))
    else:
        got = y.float().cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - want) <= acc_err + 2.0 ** -8 * np.abs(want) * 1.001)


@pytest.mark.parametrize("int8", [True, False])
@pytest.mark.parametrize("m,n,k", [(1, 64, 64), (5, 1376, 256), (5, 256, 688), (6, 1024, 256), (17, 512, 256),
                                   (8, 200, 1040), (40, 333, 2064), (72, 130, 528), (80, 96, 512), (3, 5, 16)])
def test_linear_small_and_ragged_shapes(m, n, k, int8):
    _linear_case(m, n, k, int8, residual=False, out_f32=False, seed=m * 7 + n * 3 + k)


@pytest.mark.parametrize("int8", [True, False])
def test_linear_residual_and_f32_output(int8):
    _linear_case(6, 256, 688, int8, residual=True, out_f32=False, seed=11)
    _linear_case(9, 1000, 256, int8, residual=False, out_f32=True, seed=12)
    _linear_case(9, 136, 2048, int8, residual=True, out_f32=True, seed=13)


def test_linear_exact_integer_case():
    """Integer activations and unit step sizes: every product and sum is exact in fp32, so the GPU
    must reproduce the integer result bit for bit (catches any fragment-layout slip)."""
    g = torch.Generator().manual_seed(5)
    m, n, k = 8, 192, 1024
    x = torch.randint(-4, 5, (m, k), generator=g).to(torch.bfloat16).cuda()
    q = torch.randint(-127, 128, (n, k), generator=g).to(torch.int8).cuda()
    d = torch.ones(n, dtype=torch.float32, device="cuda")
    y = binding.quasar_linear(x, q, d, out_f32=True)
    want = x.cpu().to(torch.int64) @ q.cpu().to(torch.int64).T
    assert torch.equal(y.cpu().to(torch.int64), want)


@pytest.mark.parametrize("m", [1, 4, 5, 8])
def test_linear_long_stream_with_ragged_tails_is_an_exact_integer_contraction(m):
    """Matrices of LM-head size with at most 8 rows run as an integer contraction on tcgen05 (the activations as
    three base-256 digits against a power of two above the row maximum).  With integer activations and unit step
    sizes the result must be the integer product bit for bit - on a shape whose channel count and contraction
    length both leave a partial tile - and with ordinary inputs it must agree with the oracle to fp32 rounding."""
    n, k = 33000, 4112                                  # 135.7 MB of weights; 33000 = 257 * 128 + 104, 4112 = 32 * 128 + 16
    g = torch.Generator().manual_seed(7 + m)
    x = torch.randint(-4, 5, (m, k), generator=g).to(torch.bfloat16).cuda()
    q = torch.randint(-127, 128, (n, k), generator=g, dtype=torch.int8).cuda()
    d = torch.ones(n, dtype=torch.float32, device="cuda")
    y = binding.quasar_linear(x, q, d, out_f32=True)
    rows = np.unique(np.concatenate([np.arange(0, 130), np.arange(n - 130, n), np.random.default_rng(m).integers(0, n, 256)]))
    want = x.cpu().to(torch.int64) @ q[torch.from_numpy(rows).cuda()].cpu().to(torch.int64).T
    assert torch.equal(y.cpu()[:, torch.from_numpy(rows)].to(torch.int64), want)
    # ordinary inputs, one row scaled far below the others (its digits use the same 21 bits against its own maximum)
    x = synth.normal_bf16((m, k), 1.0, seed=m, device="cuda")
    x[m - 1] = (x[m - 1].float() * 2.0 ** -20).to(torch.bfloat16)
    wq, wd = binding.quasar_quantize(synth.normal_bf16((n, k), 0.02, seed=3, device="cuda"))
    y = binding.quasar_linear(x, wq, wd, out_f32=True)
    oq = wq[torch.from_numpy(rows).cuda()].cpu().numpy()
    od = wd.cpu().numpy()[rows]
    xo = qo.bf16_bits_to_f64(_bits(x))
    want = qo.linear(xo, oq, od)
    absw = qo.linear(np.abs(xo), np.abs(oq.astype(np.int16)).astype(np.float64), od)
    got = y.cpu().numpy()[:, rows].astype(np.float64)
    assert np.all(np.abs(got - want) <= 1e-6 * absw + 2e-7 * np.abs(want))


def test_linear_is_run_to_run_identical():
    x = synth.normal_bf16((6, 4096), 1.0, seed=1, device="cuda")
    q, d = binding.quasar_quantize(synth.normal_bf16((4096, 4096), 0.02, seed=2, device="cuda"))
    ws = torch.zeros(binding.quasar_linear_workspace_bytes(6, 4096, 4096), dtype=torch.uint8, device="cuda")
    a = binding.quasar_linear(x, q, d, workspace=ws, out_f32=True).clone()
    for _ in range(3):
        b = binding.quasar_linear(x, q, d, workspace=ws, out_f32=True)
        assert torch.equal(a, b)


@pytest.mark.parametrize("k,n", [(4096, 6144), (4096, 4096), (4096, 24576), (12288, 4096), (4096, 151936)])
@pytest.mark.parametrize("m", [1, 5, 8, 40, 64])
def test_linear_qwen3_8b_shapes_sampled(k, n, m):
    x = synth.normal_bf16((m, k), 1.0, seed=m, device="cuda")
    wm = synth.normal_bf16((n, k), 0.02, seed=k + n, device="cuda")
    q, d = binding.quasar_quantize(wm)
    y = binding.quasar_linear(x, q, d, out_f32=True)
    rows = np.unique(np.concatenate([np.arange(0, 64), np.arange(n - 64, n),
                                     np.random.default_rng(n).integers(0, n, 384)]))
    oq = q[torch.from_numpy(rows).cuda()].cpu().numpy()
    od = d.cpu().numpy()[rows]
    xo = qo.bf16_bits_to_f64(_bits(x))
    want = qo.linear(xo, oq, od)
    absw = qo.linear(np.abs(xo), np.abs(oq.astype(np.int16)).astype(np.float64), od)
    got = y.cpu().numpy()[:, rows].astype(np.float64)
    assert np.all(np.abs(got - want) <= 4e-6 * absw + 1e-6 * np.abs(want))
