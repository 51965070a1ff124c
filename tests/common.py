"""Glue used by the tests: hands the same seeded bytes to the oracle and to the CUDA path."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2603_01399_b200 import synth


def master_getter(shape, seed=0, device="cpu"):
    """Returns get(kind, layer) -> bf16 torch tensor, regenerated on demand from its own sub-seed."""
    def get(kind, layer=0):
        if kind == "embed":
            return synth.embedding(shape, seed, device)
        if kind in ("attn_norm", "mlp_norm", "final_norm", "q_norm", "k_norm"):
            return synth.gain(shape, kind, layer, seed, device)
        return synth.matrix(shape, kind, layer, seed, device)
    return get


def oracle_model(shape, seed=0, int8=True, device="cpu", act_int8=False):
    get = master_getter(shape, seed, device)
    absmax = (lambda kind, layer: synth.activation_absmax(shape, kind, layer, seed).numpy()) if act_int8 else None
    return oracle.build_model(shape, lambda kind, layer: synth.bf16_bits(get(kind, layer)), int8=int8,
                              act_int8=act_int8, get_act_absmax=absmax)


def oracle_greedy_continuation(model, kv, root_token, n):
    """n greedy tokens after root_token by single-row verify calls on a scratch copy of the cache."""
    import copy
    kv2 = oracle.KVCache(kv.k_bits.copy(), kv.v_bits.copy(), kv.seq_len.copy())
    out = []
    tok = int(root_token)
    for _ in range(n):
        r = oracle.verify(model, kv2, np.array([[tok]], np.int32), None, np.array([1], np.int32))
        oracle.kv_commit(kv2, r.accept_len, None)
        tok = int(r.bonus[0])
        out.append(tok)
    return out


def prefill_oracle(model, kv, tokens_1d, chunk):
    """Push tokens through verify in chunks and commit all of them (chain blocks)."""
    toks = list(int(t) for t in tokens_1d)
    i = 0
    while i < len(toks):
        c = toks[i:i + chunk]
        t = np.array([c], np.int32)
        oracle.verify(model, kv, t, None, np.array([len(c)], np.int32), want_logits=False)
        kv.seq_len[0] += len(c)
        i += len(c)


# ---- CUDA-path side (imports nothing from oracle) ------------------------------------------
def gpu_model(shape, seed=0, int8=True, max_seq=128, gen_device="cpu", act_int8=False):
    from paper_2603_01399_b200 import binding
    absmax = (lambda kind, layer: synth.activation_absmax(shape, kind, layer, seed)) if act_int8 else None
    return binding.Model.from_master(shape, master_getter(shape, seed, gen_device), max_seq, int8=int8,
                                     act_int8=act_int8, get_act_absmax=absmax)


def logits_close(gpu, ref, abs_tol=2e-2, rel_tol=1e-2):
    """Element passes if |g - o| <= max(abs_tol, rel_tol * |o|).  Returns (ok, max_abs, max_rel)."""
    gpu = np.asarray(gpu, np.float64)
    ref = np.asarray(ref, np.float64)
    diff = np.abs(gpu - ref)
    ok = bool(np.all(diff <= np.maximum(abs_tol, rel_tol * np.abs(ref))))
    return ok, float(diff.max()), float((diff / np.maximum(np.abs(ref), 1e-30)).max())


def margins(logits):
    """top1 - top2 per row of fp32 logits [..., V]."""
    part = np.partition(logits, -2, axis=-1)
    return part[..., -1] - part[..., -2]


# ---- agreement at the benchmark's full widths -------------------------------------------------
# Every tensor of the pass is rounded to bf16 between steps, so two implementations that only ADD
# differently (fp32 instead of fp64, another summation order) drift apart through flipped roundings.
# tests/test_oracle_fullwidth_noise.py measures that drift with the oracle against itself on the CPU
# (two layers at the Qwen3-8B widths, fp32 accumulation in eight interleaved slices): 98.7 % of the
# logits inside max(2e-2, 1e-2 |o|), mean |d| 4.3e-3, worst 4.0e-2 at a logit spread of 1.33.  The
# full-width GPU tests assert the benchmark's element test on a share of the logits that leaves twice
# that many outside, and bound the mean and the worst element at 2.5 to 3 times that measured drift.
FULLWIDTH_SHARE = 0.97
FULLWIDTH_MEAN_TOL = 1.2e-2
FULLWIDTH_WORST_TOL = 1e-1


def fullwidth_stats(got, want):
    """(share of elements with |g - o| <= max(2e-2, 1e-2 |o|), mean |g - o|, worst |g - o|)."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    d = np.abs(got - want)
    return float(np.mean(d <= np.maximum(2e-2, 1e-2 * np.abs(want)))), float(d.mean()), float(d.max())
