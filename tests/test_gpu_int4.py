"""4-bit group-wise weights on the GPU against the oracle (Section 6 outlook), through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import quasar_oracle as qo
from paper_2603_01399_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _f32(t):
    return qo.bf16_bits_to_f32(synth.bf16_bits(t))


@pytest.mark.parametrize("n,k", [(5, 128), (64, 768), (1376, 256), (300, 4096), (16, 17408)])
def test_quantize_int4_bit_exact(n, k):
    w = synth.normal_bf16((n, k), 0.02, seed=n + k, device="cuda")
    w[0, :128] = 0                                       # an all-zero group
    w[min(1, n - 1), 5] = 3.0                            # an outlier inside a group
    packed, delta = binding.quasar_quantize_int4(w)
    oq, od = qo.quantize_int4(_f32(w))
    assert np.array_equal(delta.cpu().numpy().view(np.uint32), od.view(np.uint32))
    assert np.array_equal(packed.cpu().numpy(), qo.pack_int4(oq))


@pytest.mark.parametrize("m,n,k", [(1, 16, 128), (6, 200, 512), (5, 1376, 768), (17, 512, 256), (40, 300, 1024), (50, 64, 256),
                                   (6, 4096, 4096), (8, 4096, 12288)])
def test_linear_w4_matches_the_oracle(m, n, k):
    w = synth.normal_bf16((n, k), 0.02, seed=m + n + k, device="cuda")
    x = synth.normal_bf16((m, k), 1.0, seed=m * 3 + 1, device="cuda")
    packed, delta = binding.quasar_quantize_int4(w)
    y = binding.quasar_linear_w4(x, packed, delta, out_f32=True)
    codes = qo.unpack_int4(packed.cpu().numpy())
    want = qo.linear_int4(_f32(x).astype(np.float64), codes, delta.cpu().numpy())
    got = y.cpu().numpy().astype(np.float64)
    scale = np.sqrt(np.mean(want ** 2))
    assert np.all(np.abs(got - want) <= 2e-5 * np.maximum(np.abs(want), scale)), np.abs(got - want).max()   # fp32 accumulation over K terms
    # bf16 output with a residual, rounded where the decoder layer rounds; repeatable bit for bit
    res = synth.normal_bf16((m, n), 1.0, seed=9, device="cuda")
    yb = binding.quasar_linear_w4(x, packed, delta, residual=res)
    ref = qo.bf16_round(qo.bf16_round(want) + _f32(res).astype(np.float64))
    gb = yb.float().cpu().numpy().astype(np.float64)
    assert np.mean(gb != ref) < 5e-3 and np.all(np.abs(gb - ref) <= 2.0 ** -7 * np.maximum(np.abs(ref), 1e-3))
    assert torch.equal(yb, binding.quasar_linear_w4(x, packed, delta, residual=res))
