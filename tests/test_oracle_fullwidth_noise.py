"""What "agreement" can mean at the benchmark's full widths, shown on the CPU alone.

The verification pass rounds every tensor to bf16 between steps (the oracle's reading of where
tensors are rounded).  Two implementations that differ only in how they ADD - fp32 instead of
fp64, or another summation order - now and then round an element of the 4096-wide residual
stream the other way; that single step moves all 24,576 gate/up sums a little and some of
those flip in turn.  This file measures how far the oracle drifts from ITSELF when nothing but
the accumulation of its linear layers changes, at the Qwen3-8B widths (hidden 4096, 32/8 heads,
FFN 12288) with two layers and a reduced vocabulary (the statistics are per logit, so the
number of logits only has to be large).  The GPU tests at full width take their criterion from
these numbers (tests/common.py: FULLWIDTH_*), not from a comparison of GPU code with GPU code.
"""
import numpy as np
import pytest

import oracle
from oracle import quasar_oracle as qo
from paper_2603_01399_b200 import synth
from tests.common import (FULLWIDTH_MEAN_TOL, FULLWIDTH_SHARE, FULLWIDTH_WORST_TOL, fullwidth_stats, master_getter)


def _linear_fp32_sliced(x, w, delta):
    """The oracle's linear layer with nothing changed but the accumulation: fp32 partial sums over 8
    interleaved slices of the contraction index, added in slice order (what a kernel that splits K
    over eight warps does), then the step size in fp32."""
    x32 = np.asarray(x, np.float32)
    w32 = w.astype(np.float32)
    acc = np.zeros((x32.shape[0], w32.shape[0]), np.float32)
    for s in range(8):
        acc = acc + x32[:, s::8] @ w32[:, s::8].T
    if delta is not None:
        acc = acc * delta.astype(np.float32)[None, :]
    return acc.astype(np.float64)


@pytest.fixture(scope="module")
def world():
    full = synth.SHAPES["qwen3_8b"]
    shape = synth.ModelShape("qwen3_8b_2l_v16k", 2, full.hidden, full.n_q_heads, full.n_kv_heads, full.head_dim,
                             full.ffn, 16384, full.qk_norm, full.rope_theta, full.rms_eps)
    get = master_getter(shape, 0, "cpu")
    om = oracle.build_model(shape, lambda kind, layer: synth.bf16_bits(get(kind, layer)), int8=True)
    s_max = 272
    kk, vv = synth.kv_prefix(shape, 1, s_max, seed=1)
    tokens = synth.uniform_tokens((1, 6), shape.vocab, synth.sub_seed(2, "tokens")).numpy()
    bl = np.array([6], np.int32)

    def run():
        kv = oracle.KVCache(synth.bf16_bits(kk).copy(), synth.bf16_bits(vv).copy(), np.array([256], np.int32))
        return oracle.verify(om, kv, tokens, None, bl, want_trace=True)
    return run


def test_oracle_against_itself_with_another_accumulation(world, monkeypatch):
    ref = world()
    monkeypatch.setattr(qo, "linear", _linear_fp32_sliced)
    alt = world()
    monkeypatch.undo()
    again = world()
    assert np.array_equal(again.logits, ref.logits), "the oracle is deterministic"

    # the first GEMM alone: only a few roundings go the other way
    q0, q1 = ref.trace["l0.qkv.b0"], alt.trace["l0.qkv.b0"]
    first = float(np.mean(q0 != q1))
    assert 0 < first < 5e-3, first
    # two layers later the share of differing elements has grown by orders of magnitude
    x0, x1 = ref.trace["l1.x_mlp.b0"], alt.trace["l1.x_mlp.b0"]
    last = float(np.mean(x0 != x1))
    assert last > 20 * first, (first, last)

    inside, mean, worst = fullwidth_stats(alt.logits[0], ref.logits[0])
    print(f"oracle vs oracle(fp32, 8 slices): qkv flips {first:.5f}, x after 2 layers differs in {last:.3f}; "
          f"logits inside {inside:.4f}, mean |d| {mean:.3e}, worst {worst:.3e}, spread {ref.logits[0].std():.3f}")
    # The benchmark's element test (max(2e-2, 1e-2 |o|)) cannot hold for every logit even between two CPU
    # runs of the oracle's own arithmetic ...
    assert worst > 2e-2 or inside < 1.0 or mean > 1e-3
    # ... and the criterion the GPU tests use covers that drift, with a factor of about two in hand.
    assert inside >= FULLWIDTH_SHARE + (1 - FULLWIDTH_SHARE) / 3
    assert mean <= 0.6 * FULLWIDTH_MEAN_TOL
    assert worst <= 0.6 * FULLWIDTH_WORST_TOL
    # (and it is not slack either: the drift is within a factor of four of every bound)
    assert (1 - inside) >= (1 - FULLWIDTH_SHARE) / 4 and mean >= FULLWIDTH_MEAN_TOL / 4 and worst >= FULLWIDTH_WORST_TOL / 4
    # top-1 only moves on rows whose top-2 margin is inside the drift
    part = np.partition(ref.logits[0], -2, axis=-1)
    margin = part[:, -1] - part[:, -2]
    safe = margin > 2 * worst
    assert np.array_equal(alt.logits[0].argmax(-1)[safe], ref.logits[0].argmax(-1)[safe])
