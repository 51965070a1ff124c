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
