"""The allocation-free linear layer (quasar_linear_static) against quasar_linear (needs a GPU).

Some hosts of this library may not call cudaMalloc at all (a plug-in whose host application owns
the memory pool, or a serving loop that keeps the allocator out of its critical path), so they have
no workspace to pass.  quasar_linear_static takes its split-K scratch from a fixed array inside the
library instead.  It must give exactly what quasar_linear gives, call after call, although every
call finds the previous call's leftovers in that array.  The file name makes pytest collect it last.
"""
import pytest
import torch

from paper_2603_01399_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _case(m, n, k, seed, int8=True, out_f32=True, residual=False):
    x = synth.normal_bf16((m, k), 1.0, seed=seed, device="cuda")
    wm = synth.normal_bf16((n, k), 0.02, seed=seed + 1, device="cuda")
    res = synth.normal_bf16((m, n), 1.0, seed=seed + 2, device="cuda") if residual else None
    if int8:
        w, d = binding.quasar_quantize(wm)
    else:
        w, d = wm, None
    want = binding.quasar_linear(x, w, d, residual=res, out_f32=out_f32)
    out = torch.full((m, n), float("nan"), dtype=torch.float32 if out_f32 else torch.bfloat16, device="cuda")
    return x, w, d, res, want, out


def test_two_calls_in_a_row_match_the_workspace_version():
    # both shapes split the contraction over several CTAs, so the scratch array is really used; the
    # second call has a different split and finds the first call's partial sums and counters in it
    for m, n, k, seed in ((6, 4096, 4096, 21), (5, 1376, 2064, 22)):
        assert binding.quasar_linear_workspace_bytes(m, n, k) > 4096
        x, w, d, res, want, out = _case(m, n, k, seed)
        binding.quasar_linear_static(x, w, d, out)
        torch.cuda.synchronize()
        # the split-K sum runs in a fixed order in both entry points: the results are identical, which
        # is inside every tolerance the other linear tests use
        assert torch.equal(out, want)
    # the same shape twice, bf16 output with a residual, bf16 weights
    x, w, d, res, want, out = _case(8, 512, 4096, 23, int8=False, out_f32=False, residual=True)
    for _ in range(2):
        out.fill_(float("nan"))
        binding.quasar_linear_static(x, w, d, out, residual=res)
        torch.cuda.synchronize()
        assert torch.equal(out, want)


def test_a_warmed_up_call_allocates_nothing_and_blocks_of_more_than_72_rows_work():
    """The point of the entry: after its first call on the device (which looks the array up) a call leaves
    the device's free memory exactly as it found it; and a block of 80 rows takes the same route."""
    x, w, d, res, want, out = _case(80, 256, 512, 31)
    binding.quasar_linear_static(x, w, d, out)                      # first call: address lookup
    torch.cuda.synchronize()
    assert torch.equal(out, want)
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        binding.quasar_linear_static(x, w, d, out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert torch.equal(out, want)


def test_refuses_shapes_beyond_the_built_in_scratch():
    cap = binding.quasar_linear_static_scratch_bytes()
    assert cap == 4 << 20
    m, n, k = 64, 24576, 4096
    assert binding.quasar_linear_workspace_bytes(m, n, k) > cap
    x = torch.zeros((m, k), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((n, k), dtype=torch.int8, device="cuda")
    d = torch.ones(n, dtype=torch.float32, device="cuda")
    out = torch.zeros((m, n), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.QuasarError) as e:
        binding.quasar_linear_static(x, w, d, out)
    assert e.value.code == -3 and "scratch" in str(e.value)


def test_a_very_large_matrix_with_few_rows_still_fits_the_built_in_scratch():
    """With a workspace, blocks of at most 8 rows on matrices of LM-head size take a kernel that needs several MB of
    scratch; without one the call must fall back to the kernel that needs none for this shape, not refuse it."""
    m, n, k = 6, 33000, 4112
    x = synth.normal_bf16((m, k), 1.0, seed=3, device="cuda")
    q, d = binding.quasar_quantize(synth.normal_bf16((n, k), 0.02, seed=4, device="cuda"))
    out = torch.zeros((m, n), dtype=torch.float32, device="cuda")
    binding.quasar_linear_static(x, q, d, out)
    want = binding.quasar_linear(x, q, d, out_f32=True)      # (the stream kernel: sums exact integers, so not bit-equal)
    torch.cuda.synchronize()
    assert torch.all((out - want).abs() <= 1e-5 * want.abs() + 3e-4)      # fp32 accumulation of 4112 terms of size ~0.02
