#!/usr/bin/env python
"""Benchmark of the quantised verification pass (Quasar, arXiv 2603.01399) on B200.

One "step" = one whole verify pass (embedding -> 36 decoder layers with int8 weights -> LM head
-> arg-max -> greedy acceptance) of the Qwen3-8B-shaped workload: batch 1, 1024 cached positions,
chain draft of 5 (6 block rows).  Inputs are seeded and synthetic (random-init weights of that
architecture, N(0,1) KV prefix, the bf16 model's greedy continuation corrupted with p = 0.3 as
the draft); they stand in for the paper's Qwen3-8B runs on Spec-Bench style prompts.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `--impl reference` times the CPU oracle (the plain fp64 restatement the
tests compare against) on the host cores, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2603_01399_b200 import synth  # noqa: E402

WORKLOAD = "qwen3-8b-shaped verify pass: B=1, prefix 1024, chain draft gamma=5 (6 block rows), int8 weights"
PREFIX, GAMMA, BATCH = 1024, 5, 1
METRIC = "verify-pass latency & accepted tok/s, Qwen3-8B shape; HBM GB/s as % of peak"
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the persistent kernel on the 2-layer case
# of `--profile-pass --profile-layers 2` (the ncu capture summarised in profiles/), and that case's
# algorithmic bytes.  Traffic follows the weight bytes, so a full launch is taken as the same ratio times
# its own algorithmic bytes.  Both None while the kernel has changed since that capture.
NCU_CASE_DRAM_BYTES = 1_017_723_000 + 7_401_472
NCU_CASE_ALGORITHMIC_BYTES = 1_017_652_736
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


def algorithmic_bytes(shape, batch, t_rows, prefix_total, weight_bytes_per_elem):
    """Bytes one verify pass has to move (Section 3.4's M * bytes / BW term plus the KV stream)."""
    w = shape.weight_elems() * weight_bytes_per_elem
    n_out = sum(n for _, n, _ in shape.linear_shapes()[:4]) * shape.n_layers + shape.vocab
    scales = n_out * 4 if weight_bytes_per_elem == 1 else 0
    m = batch * t_rows
    kv_read = shape.n_layers * prefix_total * shape.n_kv_heads * shape.head_dim * 2 * 2
    kv_write = shape.n_layers * m * shape.n_kv_heads * shape.head_dim * 2 * 2
    embed = m * shape.hidden * 2
    gains = (2 * shape.n_layers + 1) * shape.hidden * 2
    return {"weights": w, "scales": scales, "kv_read": kv_read, "kv_write": kv_write, "embed": embed,
            "gains": gains, "total": w + scales + kv_read + kv_write + embed + gains}


def max_over_ranks(value: float, dist, device) -> float:
    """The slowest rank's time: replicas are independent, so the job is as slow as its slowest GPU."""
    if dist is None:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def sum_over_ranks(value: float, dist, device) -> float:
    """Units processed by the whole job (every replica works on its own sequences)."""
    if dist is None:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t[0])


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 7 and r[3 + i] == "Active" for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def master_getter(shape, seed, device):
    cache = {}

    def get(kind, layer=0):
        if kind == "embed":
            if "embed" not in cache:
                cache["embed"] = synth.embedding(shape, seed, device)
            return cache["embed"]
        if kind in ("attn_norm", "mlp_norm", "final_norm", "q_norm", "k_norm"):
            return synth.gain(shape, kind, layer, seed, device)
        return synth.matrix(shape, kind, layer, seed, device)
    return get


def greedy_continuation(binding, model, kv, root, n):
    """n greedy tokens of `model` after `root`, by plain decode steps on a scratch copy of the cache."""
    scratch = binding.KVCache(model.shape, kv.batch, kv.s_max, k=kv.k.clone(), v=kv.v.clone(),
                              seq_len=kv.seq_len.clone())
    buf = binding.VerifyBuffers(model, kv.batch, 1, want_logits=False)
    tok = root.clone()
    out = []
    for _ in range(n):
        buf.tokens.copy_(tok.view(-1, 1))
        binding.quasar_verify(model, scratch, buf)
        binding.quasar_kv_commit(model, scratch, buf)
        tok = buf.bonus.clone()
        out.append(tok.clone())
    torch.cuda.synchronize()
    return torch.stack(out, dim=1)      # [B][n]


# ------------------------------------------------------------------------------------------
def run_ours(args):
    from paper_2603_01399_b200 import binding, build
    build.build()
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    shape = synth.SHAPES["qwen3_8b"]
    t_rows = GAMMA + 1
    s_max = PREFIX + 16
    get = master_getter(shape, 0, "cuda")
    m_int8 = binding.Model.from_master(shape, get, 4096 + 16, int8=True)   # (the batch-of-eight line below has prefixes up to 4096)
    m_bf16 = binding.Model.from_master(shape, get, s_max, int8=False)
    kk, vv = synth.kv_prefix(shape, BATCH, s_max, seed=1, device="cuda")
    kv = binding.KVCache(shape, BATCH, s_max, k=kk, v=vv,
                         seq_len=torch.full((BATCH,), PREFIX, dtype=torch.int32, device="cuda"))
    root = synth.uniform_tokens((BATCH,), shape.vocab, synth.sub_seed(2, "tokens")).cuda()
    greedy = greedy_continuation(binding, m_bf16, kv, root, GAMMA)
    draft = synth.corrupt_draft(greedy, 0.3, shape.vocab, seed=2)
    tokens_host = torch.cat([root.cpu().view(-1, 1), draft], dim=1).to(torch.int32).contiguous().pin_memory()

    def timed_plan(model, steps, warmup, sample_clocks):
        buf = binding.VerifyBuffers(model, BATCH, t_rows, want_logits=False)
        buf.tokens.copy_(tokens_host)
        plan = binding.Plan(model, kv, buf)
        for _ in range(warmup):
            plan.launch()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        sampler = ClockSampler(local) if sample_clocks else None
        if sampler:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = binding.kernel_launches()
        torch.cuda.synchronize()
        if sample_clocks:
            torch.cuda.profiler.start()      # lets `ncu --profile-from-start off` list the timed launches only
        e0.record()
        for _ in range(steps):
            plan.launch()
        e1.record()
        torch.cuda.synchronize()
        if sample_clocks:
            torch.cuda.profiler.stop()
        launches = binding.kernel_launches() - l0
        clocks = sampler.stop() if sampler else None
        if dist is not None:
            dist.barrier()
        ms = max_over_ranks(e0.elapsed_time(e1), dist, "cuda")
        return ms / steps, buf, plan, launches, clocks

    ms_step, buf, plan, launches, clocks = timed_plan(m_int8, args.steps, args.warmup, True)
    accepted = int((buf.accept_len + 1).sum())            # accepted drafts + the bonus token, per pass
    accepted_drafts = int(buf.accept_len.sum())
    status = int(buf.status[0])

    # end to end: host tokens in, host decision out, every step
    al = torch.zeros(BATCH, dtype=torch.int32).pin_memory()
    bo = torch.zeros(BATCH, dtype=torch.int32).pin_memory()
    for _ in range(3):
        plan.run_host(tokens_host, al, bo)
    if dist is not None:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        plan.run_host(tokens_host, al, bo)
    e2e_ms = max_over_ranks((time.perf_counter() - t0) * 1e3 / args.steps, dist, "cuda")
    accepted_job = sum_over_ranks(accepted, dist, "cuda")          # every replica verifies its own sequences
    accepted_drafts_job = sum_over_ranks(accepted_drafts, dist, "cuda")

    # Random-initialised int8 and bf16 weights do not share their arg-max, so the bf16 model's draft is
    # rarely accepted.  Beside it: the same pass on a draft that is the int8 model's own greedy continuation
    # with the same replacement probability (the pass costs the same whatever the tokens are).
    own = synth.corrupt_draft(greedy_continuation(binding, m_int8, kv, root, GAMMA), 0.3, shape.vocab, seed=2)
    sbuf = binding.VerifyBuffers(m_int8, BATCH, t_rows, want_logits=False)
    sbuf.tokens.copy_(torch.cat([root.cpu().view(-1, 1), own], dim=1).to(torch.int32))
    binding.quasar_verify(m_int8, kv, sbuf)
    torch.cuda.synchronize()
    own_accepted = sum_over_ranks(int((sbuf.accept_len + 1).sum()), dist, "cuda")

    # latency distribution: 100 more replays, each between its own pair of events
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(100)]
    for a, b in evs:
        a.record()
        plan.launch()
        b.record()
    torch.cuda.synchronize()
    lat = sorted(a.elapsed_time(b) for a, b in evs)
    lat_median, lat_min = lat[len(lat) // 2], lat[0]

    # how far the int8 model is from its bf16 sibling on this block (random weights; no pass/fail):
    # top-1 agreement over the block rows and the mean logit difference in units of the logit spread
    cmp_logits = {}
    for name, model in (("int8", m_int8), ("bf16", m_bf16)):
        lb = binding.VerifyBuffers(model, BATCH, t_rows, want_logits=True)
        lb.tokens.copy_(tokens_host)
        binding.quasar_verify(model, kv, lb)
        torch.cuda.synchronize()
        cmp_logits[name] = lb.logits.float()
        del lb
    agree = float((cmp_logits["int8"].argmax(-1) == cmp_logits["bf16"].argmax(-1)).float().mean())
    rel_diff = float((cmp_logits["int8"] - cmp_logits["bf16"]).abs().mean() / cmp_logits["bf16"].std())
    del cmp_logits

    peaks, peak_kind = measured_peaks()
    hbm_peak = float(peaks["hbm_gbs"])
    batch8 = time_batch8(binding, m_int8, shape, max(3, args.steps // 5), hbm_peak) if rank == 0 else None

    # the per-step skinny GEMM (used for blocks of more than 8 rows) over the model's 145 matrices in pass order
    gemm = time_gemm_sweep(binding, m_int8, shape, BATCH * t_rows, max(3, args.steps // 4))

    # bf16-weight sibling pass (the "BF16 verifier" of Section 3.4, same kernels)
    bf16_ms, bbuf, bplan, _, _ = timed_plan(m_bf16, max(3, args.steps // 4), 3, False)
    bplan.close()
    del bbuf, bplan
    m_bf16.close()
    del m_bf16
    torch.cuda.empty_cache()
    extra = {}
    if rank == 0 and not args.headline_only:
        extra["gamma_sweep"] = gamma_sweep(binding, m_int8, shape, kv, root, hbm_peak)
        extra["int4_linear"] = int4_linear_line(binding, hbm_peak)
        extra["w8a8"] = time_w8a8(binding, shape, kv, tokens_host, max(3, args.steps // 4), hbm_peak)
        extra["linear_sweep"] = linear_sweep_summary(binding, hbm_peak)
        extra["tree14b"] = time_tree14b(binding, max(3, args.steps // 5), hbm_peak)

    ab = algorithmic_bytes(shape, BATCH, t_rows, PREFIX * BATCH, 1)
    ab16 = algorithmic_bytes(shape, BATCH, t_rows, PREFIX * BATCH, 2)
    pass_gbs = ab["total"] / (ms_step * 1e-3) / 1e9
    # roofline of the dominant kernel: the persistent verify kernel, one launch per step, so its average
    # launch duration is the step time measured above with CUDA events on the launching stream
    launch_gbs = ab["total"] / (ms_step * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": accepted_job / (ms_step * 1e-3),
        "unit": "accepted tok/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8 weights, f16 mma operands, f32 accumulate",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "replicas": world, "batch": BATCH, "prefix": PREFIX, "gamma": GAMMA,
                   "l2": "inputs (7.7 GB of weights + KV per pass) exceed the 126 MB L2; no flush needed",
                   "launch": "one persistent cooperative kernel per step"},
        "verify_latency_ms": ms_step, "verify_latency_ms_median_of_100": lat_median, "verify_latency_ms_min_of_100": lat_min,
        "int8_vs_bf16": {"top1_agreement": agree, "mean_abs_logit_diff_over_logit_std": rel_diff,
                         "note": "random-initialised weights: quantisation noise through 36 random layers decorrelates the logits"},
        "batch8_ragged": batch8, **extra,
        "accepted_per_pass": accepted, "accepted_drafts_per_pass": accepted_drafts,
        "accepted_drafts_tok_s": accepted_drafts_job / (ms_step * 1e-3), "device_status": status,
        "own_draft": {"what": "draft = the int8 model's own greedy continuation, each token replaced w.p. 0.3",
                      "accepted_per_pass": own_accepted / world, "accepted_tok_s": own_accepted / (ms_step * 1e-3)},
        "pass_bytes": ab, "pass_hbm_gbs": pass_gbs, "pass_hbm_frac_of_measured_copy": pass_gbs / hbm_peak,
        "pass_hbm_frac_of_nominal_8TBs": pass_gbs / NOMINAL_HBM_GBS,
        "bf16_sibling": {"verify_latency_ms": bf16_ms, "ratio_vs_int8": bf16_ms / ms_step,
                         "pass_hbm_gbs": ab16["total"] / (bf16_ms * 1e-3) / 1e9},
        "per_step_gemm_sweep": {"kernel": "quasar_linear at 6 rows over the 145 matrices of a pass (skinny_gemm_kernel; LM head: umma_stream_kernel), one CUDA graph", "gbs": gemm["gbs"], "avg_launch_us": gemm["avg_us"]},
        "clocks": clocks,
        "e2e": {"value": accepted_job / (e2e_ms * 1e-3), "unit": "accepted tok/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": tokens_host.numel() * 4, "d2h_bytes_per_step": 2 * BATCH * 4},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "verify_megakernel<int8, 128> (persistent, one launch per step)",
                     "achieved": launch_gbs, "peak": hbm_peak, "unit": "GB/s", "frac": launch_gbs / hbm_peak,
                     "peak_kind": f"{peak_kind} copy bandwidth", "traffic": (round(ab["total"] * NCU_CASE_DRAM_BYTES / NCU_CASE_ALGORITHMIC_BYTES)
                                 if NCU_CASE_DRAM_BYTES else None),
                     "traffic_source": "ncu dram bytes of a 2-of-36-layer launch x (algorithmic bytes of this launch / of that one)",
                     "avg_launch_us": ms_step * 1e3, "bytes_per_launch": ab["total"]},
    }
    if rank == 0:
        out["cpu_baseline"] = cpu_baseline(shape, accepted)
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def time_batch8(binding, model, shape, reps, hbm_peak):
    """Not the headline: the same model on 8 sequences with seeded prefixes in 512..4096 and chains of 8
    drafts (72 block rows), which runs one kernel per step (a CUDA graph).  Latency and bytes only."""
    import numpy as np
    rng = np.random.default_rng(4)
    prefix = [int(x) for x in rng.integers(512, 4097, 8)]
    s_max = 4096 + 16
    kk, vv = synth.kv_prefix(shape, 8, s_max, seed=1, device="cuda")
    kv = binding.KVCache(shape, 8, s_max, k=kk, v=vv, seq_len=torch.tensor(prefix, dtype=torch.int32, device="cuda"))
    buf = binding.VerifyBuffers(model, 8, 9, want_logits=False)
    buf.tokens.copy_(synth.uniform_tokens((8, 9), shape.vocab, synth.sub_seed(2, "tokens")))
    plan = binding.Plan(model, kv, buf)
    for _ in range(3):
        plan.launch()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        plan.launch()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    ab = algorithmic_bytes(shape, 8, 9, sum(prefix), 1)
    gbs = ab["total"] / (ms * 1e-3) / 1e9
    out = {"workload": "B=8, prefixes U(512,4096) (sum %d), chain gamma=8, 72 block rows, int8 weights" % sum(prefix),
           "verify_latency_ms": ms, "pass_bytes": ab["total"], "pass_hbm_gbs": gbs,
           "roofline": {"bound": "hbm", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gbs / hbm_peak},
           "launch": "one kernel per step, replayed as a CUDA graph", "device_status": int(buf.status[0])}
    plan.close()
    del kv, buf, kk, vv
    return out


def _time_plan(plan, reps, warm=3):
    for _ in range(warm):
        plan.launch()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        plan.launch()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def time_tree14b(binding, reps, hbm_peak):
    """Not the headline: the Qwen3-14B-shaped model (40 layers, hidden 5120, 40/8 heads, FFN 17408), B=4,
    2048 cached positions, the 16-node draft tree (17 rows per sequence, 68 block rows), int8 weights."""
    shape = synth.SHAPES["qwen3_14b"]
    s_max = 2048 + 32
    model = binding.Model.from_master(shape, master_getter(shape, 0, "cuda"), s_max, int8=True)
    kk, vv = synth.kv_prefix(shape, 4, s_max, seed=1, device="cuda")
    kv = binding.KVCache(shape, 4, s_max, k=kk, v=vv, seq_len=torch.full((4,), 2048, dtype=torch.int32, device="cuda"))
    buf = binding.VerifyBuffers(model, 4, 17, want_logits=False, tree=True)
    buf.tokens.copy_(synth.uniform_tokens((4, 17), shape.vocab, synth.sub_seed(2, "tokens")))
    buf.parents.copy_(torch.tensor([synth.tree_parents_16()] * 4, dtype=torch.int32))
    plan = binding.Plan(model, kv, buf)
    ms = _time_plan(plan, reps)
    ab = algorithmic_bytes(shape, 4, 17, 4 * 2048, 1)
    gbs = ab["total"] / (ms * 1e-3) / 1e9
    out = {"workload": "qwen3-14b-shaped, B=4, prefix 2048, tree of 16 nodes (17 rows per sequence, 68 block rows), int8 weights",
           "verify_latency_ms": ms, "pass_bytes": ab["total"], "pass_hbm_gbs": gbs,
           "accepted_per_pass": int((buf.accept_len + 1).sum()),
           "roofline": {"bound": "hbm", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gbs / hbm_peak},
           "launch": "one kernel per step, replayed as a CUDA graph", "device_status": int(buf.status[0])}
    plan.close()
    model.close()
    del model, kv, buf, kk, vv
    torch.cuda.empty_cache()
    return out


def time_w8a8(binding, shape, kv, tokens_host, reps, hbm_peak):
    """The paper's W8A8 verifier (Section 3.2-3.3) on the headline workload: smoothing factors from synthetic
    calibration maxima, int8 activations per token, integer tensor-core GEMMs."""
    model = binding.Model.from_master(shape, master_getter(shape, 0, "cuda"), 4096 + 16, int8=True, act_int8=True,
                                      get_act_absmax=lambda kind, layer: synth.activation_absmax(shape, kind, layer, 0, "cuda"))
    buf = binding.VerifyBuffers(model, BATCH, GAMMA + 1, want_logits=False)
    buf.tokens.copy_(tokens_host)
    plan = binding.Plan(model, kv, buf)
    ms = _time_plan(plan, reps)
    ab = algorithmic_bytes(shape, BATCH, GAMMA + 1, PREFIX * BATCH, 1)
    smooth = (2 * shape.hidden + shape.q_dim + shape.ffn) * 4 * shape.n_layers + shape.hidden * 4
    total = ab["total"] + smooth
    gbs = total / (ms * 1e-3) / 1e9
    out = {"workload": WORKLOAD.replace("int8 weights", "int8 weights and int8 activations (W8A8, smoothed)"),
           "verify_latency_ms": ms, "pass_bytes": total, "pass_hbm_gbs": gbs,
           "accepted_per_pass": int((buf.accept_len + 1).sum()),
           "roofline": {"bound": "hbm", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gbs / hbm_peak},
           "launch": model.launch_kind(BATCH, GAMMA + 1), "device_status": int(buf.status[0])}
    plan.close()
    # the batch-of-eight workload with the same W8A8 model (72 block rows: tcgen05 kind::i8 linear layers)
    b8 = time_batch8(binding, model, shape, max(3, reps // 2), hbm_peak)
    b8["workload"] = b8["workload"].replace("int8 weights", "int8 weights and int8 activations (W8A8, smoothed)")
    out["batch8_ragged"] = b8
    model.close()
    del model, buf
    torch.cuda.empty_cache()
    return out


def linear_sweep_summary(binding, hbm_peak):
    """Compact form of `--linear-sweep` for the bench line: int8 weights, the five Qwen3-8B matrix shapes, row
    counts 1..64; per shape the best and the worst cell as a fraction of the copy bandwidth.  Distinct weight
    copies (>= 1 GB in total) per cell so that no launch finds its matrix in L2."""
    shapes = [("qkv", 4096, 6144), ("o", 4096, 4096), ("gateup", 4096, 24576), ("down", 12288, 4096), ("lm_head", 4096, 151936)]
    rows = [1, 2, 4, 5, 8, 16, 40, 64]
    out = {}
    for name, k, n in shapes:
        copies = max(2, -(-(1 << 30) // (n * k)))
        master = synth.normal_bf16((n, k), 0.02, seed=k + n, device="cuda")
        q, d = binding.quasar_quantize(master)
        ws_list = [q] + [q.clone() for _ in range(copies - 1)]
        cells = {}
        for m in rows:
            x = synth.normal_bf16((m, k), 1.0, seed=m, device="cuda")
            y = torch.empty((m, n), dtype=torch.bfloat16, device="cuda")
            ws = torch.zeros(binding.quasar_linear_workspace_bytes(m, n, k), dtype=torch.uint8, device="cuda")
            for w in ws_list:
                binding.quasar_linear(x, w, d, workspace=ws, out=y)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(2):
                for w in ws_list:
                    binding.quasar_linear(x, w, d, workspace=ws, out=y)
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / (2 * copies)
            cells[m] = (n * k + 4 * n) / (us * 1e-6) / 1e9 / hbm_peak
        best, worst = max(cells, key=cells.get), min(cells, key=cells.get)
        out[name] = {"K": k, "N": n, "best": {"M": best, "frac": cells[best]}, "worst": {"M": worst, "frac": cells[worst]},
                     "frac_by_rows": {str(m): round(f, 4) for m, f in cells.items()}}
        del ws_list, master, q
        torch.cuda.empty_cache()
    return {"what": "quantised linear layer alone (quasar_linear, int8 weights), fraction of the measured copy bandwidth",
            "shapes": out}


def gamma_sweep(binding, model, shape, kv, root, hbm_peak):
    """Section 4.4 / Table 3 and Eq. 13 in miniature: verify latency and accepted tokens per second against the
    draft length gamma, on the model's own greedy continuation with each token replaced w.p. 0.3, plus the cost
    of the prompt-lookup drafter on a 4096-token history (T_draft of Eq. 13)."""
    out = {}
    greedy = greedy_continuation(binding, model, kv, root, 9)
    for gamma in (3, 5, 7, 9):
        draft = synth.corrupt_draft(greedy[:, :gamma], 0.3, shape.vocab, seed=2)
        buf = binding.VerifyBuffers(model, BATCH, gamma + 1, want_logits=False)
        buf.tokens.copy_(torch.cat([root.cpu().view(-1, 1), draft], dim=1).to(torch.int32))
        plan = binding.Plan(model, kv, buf)
        ms = _time_plan(plan, 10)
        acc = int((buf.accept_len + 1).sum())
        out[str(gamma)] = {"verify_latency_ms": ms, "accepted_per_pass": acc, "accepted_tok_s": acc / (ms * 1e-3),
                           "launch": model.launch_kind(BATCH, gamma + 1)}
        plan.close()
        del buf
    hist = synth.uniform_tokens((BATCH, 4096), 50, synth.sub_seed(3, "tokens")).cuda()
    hlen = torch.full((BATCH,), 4096, dtype=torch.int32, device="cuda")
    binding.quasar_ngram_draft(hist, hlen, 5, 1, 4)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(20):
        binding.quasar_ngram_draft(hist, hlen, 5, 1, 4)
    e1.record()
    torch.cuda.synchronize()
    out["ngram_draft_us"] = e0.elapsed_time(e1) * 1e3 / 20
    return out


def int4_linear_line(binding, hbm_peak):
    """The 4-bit group-wise linear layer alone on the gate+up shape at 6 rows, distinct weight copies per launch."""
    k, n, m = 4096, 24576, 6
    master = synth.normal_bf16((n, k), 0.02, seed=k + n, device="cuda")
    packed, delta = binding.quasar_quantize_int4(master)
    copies = 24
    plist = [packed] + [packed.clone() for _ in range(copies - 1)]
    x = synth.normal_bf16((m, k), 1.0, seed=m, device="cuda")
    y = torch.empty((m, n), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(1 << 26, dtype=torch.uint8, device="cuda")
    for p in plist:
        binding.quasar_linear_w4(x, p, delta, workspace=ws, out=y)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(3):
        for p in plist:
            binding.quasar_linear_w4(x, p, delta, workspace=ws, out=y)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (3 * copies)
    nbytes = n * k // 2 + n * (k // 128) * 4
    return {"what": "quasar_linear_w4, gate+up shape (K 4096, N 24576), 6 rows", "us_per_launch": us, "bytes": nbytes,
            "gbs": nbytes / (us * 1e-6) / 1e9, "frac": nbytes / (us * 1e-6) / 1e9 / hbm_peak}


def run_linear_sweep(args):
    """`--linear-sweep`: the quantised linear layer alone over the Qwen3-8B matrix shapes and row counts,
    int8 and bf16 weights.  Every cell cycles through distinct weight copies (>= 2 GB in total) inside one
    CUDA graph, so that no launch finds its matrix in L2.  One JSON line per cell; nothing here is the
    benchmark value."""
    from paper_2603_01399_b200 import binding, build
    build.build()
    torch.cuda.set_device(0)
    peaks, peak_kind = measured_peaks()
    hbm_peak = float(peaks["hbm_gbs"])
    shapes = [(4096, 6144), (4096, 4096), (4096, 24576), (12288, 4096), (4096, 151936)]
    rows = [1, 2, 4, 5, 8, 16, 40, 64]
    for k, n in shapes:
        for int8 in (True, False):
            per = n * k * (1 if int8 else 2)
            copies = max(2, -(-(2 << 30) // per))
            master = synth.normal_bf16((n, k), 0.02, seed=k + n, device="cuda")
            if int8:
                q, d = binding.quasar_quantize(master)
                ws_list = [q] + [q.clone() for _ in range(copies - 1)]
            else:
                d = None
                ws_list = [master] + [master.clone() for _ in range(copies - 1)]
            for m in rows:
                x = synth.normal_bf16((m, k), 1.0, seed=m, device="cuda")
                y = torch.empty((m, n), dtype=torch.bfloat16, device="cuda")
                ws = torch.zeros(binding.quasar_linear_workspace_bytes(m, n, k), dtype=torch.uint8, device="cuda")

                def sweep():
                    for w in ws_list:
                        binding.quasar_linear(x, w, d, workspace=ws, out=y)
                sweep()
                torch.cuda.synchronize()
                stream = torch.cuda.Stream()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.stream(stream):
                    with torch.cuda.graph(graph, stream=stream):
                        sweep()
                    graph.replay()
                    torch.cuda.synchronize()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    for _ in range(3):
                        graph.replay()
                    e1.record(stream)
                torch.cuda.synchronize()
                us = e0.elapsed_time(e1) * 1e3 / (3 * copies)
                nbytes = per + (n * 4 if int8 else 0)
                print(json.dumps({"linear_sweep": True, "K": k, "N": n, "M": m, "weights": "int8" if int8 else "bf16",
                                  "us_per_launch": us, "gbs": nbytes / (us * 1e-6) / 1e9,
                                  "frac_of_%s_copy_bw" % peak_kind: nbytes / (us * 1e-6) / 1e9 / hbm_peak,
                                  "distinct_weight_copies": copies}), flush=True)
                del graph
            del ws_list, master


def time_gemm_sweep(binding, model, shape, m_rows, reps):
    """All GEMM launches of one pass, back to back, between two events on the launching stream."""
    t = model.tensors
    x_h = synth.normal_bf16((m_rows, shape.hidden), 1.0, 5, "cuda")
    x_q = synth.normal_bf16((m_rows, shape.q_dim), 1.0, 6, "cuda")
    x_f = synth.normal_bf16((m_rows, shape.ffn), 1.0, 7, "cuda")
    outs = {n: torch.empty((m_rows, n), dtype=torch.bfloat16, device="cuda")
            for n in (shape.qkv_dim, shape.hidden, 2 * shape.ffn)}
    logits = torch.empty((m_rows, shape.vocab), dtype=torch.float32, device="cuda")
    ws = torch.zeros(model.workspace_bytes(BATCH, m_rows // BATCH), dtype=torch.uint8, device="cuda")
    jobs = []
    for l in range(shape.n_layers):
        jobs += [(x_h, t[f"l{l}.qkv_w"], t[f"l{l}.qkv_delta"], outs[shape.qkv_dim], False),
                 (x_q, t[f"l{l}.o_w"], t[f"l{l}.o_delta"], outs[shape.hidden], False),
                 (x_h, t[f"l{l}.gateup_w"], t[f"l{l}.gateup_delta"], outs[2 * shape.ffn], False),
                 (x_f, t[f"l{l}.down_w"], t[f"l{l}.down_delta"], outs[shape.hidden], False)]
    jobs.append((x_h, t["lm_w"], t["lm_delta"], logits, True))
    nbytes = sum(j[1].numel() + j[2].numel() * 4 for j in jobs)

    def sweep():
        for x, w, d, y, f32 in jobs:
            binding.quasar_linear(x, w, d, out_f32=f32, workspace=ws, out=y)
    sweep()
    torch.cuda.synchronize()
    # replayed as one CUDA graph so that host launch cost does not enter the kernel's time
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            sweep()
        graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            graph.replay()
        e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    return {"gbs": nbytes / (ms * 1e-3) / 1e9, "avg_us": ms * 1e3 / len(jobs), "bytes_per_launch": nbytes / len(jobs),
            "launches": len(jobs)}


# ------------------------------------------------------------------------------------------
class OracleSample:
    """The CPU oracle on a bounded sample of the workload: ONE decoder layer (with the 1024-position KV
    prefix) and the LM head, at the full Qwen3-8B widths.  Built once; `time_once` runs the sample and
    returns the pass time extrapolated to all layers."""

    def __init__(self, shape):
        import oracle
        self.oracle, self.shape = oracle, shape
        small = synth.ModelShape("sample", 1, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                                 shape.ffn, shape.vocab, shape.qk_norm, shape.rope_theta, shape.rms_eps)
        get = master_getter(small, 0, "cpu")
        self.om = oracle.build_model(small, lambda kind, layer: synth.bf16_bits(get(kind, layer)), int8=True)
        kk, vv = synth.kv_prefix(small, BATCH, PREFIX + 16, seed=1)
        self.okv = oracle.KVCache(synth.bf16_bits(kk), synth.bf16_bits(vv), np.full(BATCH, PREFIX, np.int32))
        self.toks = synth.uniform_tokens((BATCH, GAMMA + 1), shape.vocab, synth.sub_seed(2, "tokens")).numpy()
        self.bl = np.full(BATCH, GAMMA + 1, np.int32)
        try:
            from threadpoolctl import threadpool_info
            self.threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        except Exception:
            self.threads = os.cpu_count() or 1

    def time_once(self):
        t0 = time.perf_counter()
        self.oracle.verify(self.om, self.okv, self.toks, None, self.bl, n_layers_run=0)
        head = time.perf_counter() - t0
        t0 = time.perf_counter()
        self.oracle.verify(self.om, self.okv, self.toks, None, self.bl, want_logits=False)
        per_layer = time.perf_counter() - t0
        return per_layer, head, per_layer * self.shape.n_layers + head


def cpu_baseline(shape, accepted):
    sample = OracleSample(shape)
    per_layer, head, full = sample.time_once()
    return {"value": accepted / full, "unit": "accepted tok/s", "cores": sample.threads, "kind": "oracle",
            "sample": f"1 of {shape.n_layers} decoder layers ({per_layer:.2f} s) + LM head and acceptance ({head:.2f} s) "
                      f"at full Qwen3-8B widths, B=1, prefix 1024, 6 block rows; scaled to {shape.n_layers} layers "
                      f"= {full:.1f} s per pass",
            "seconds_per_pass_extrapolated": full, "host_cpus": os.cpu_count()}


def run_reference(args):
    """The reference arm: the CPU oracle as it stands, on the host cores (rank 0 only).  A step is the
    bounded sample above (one decoder layer + the LM head at full widths), scaled to the 36 layers."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    shape = synth.SHAPES["qwen3_8b"]
    sample = OracleSample(shape)
    times, sampled = [], []
    for i in range(args.warmup + args.steps):
        per_layer, head, full = sample.time_once()
        if i >= args.warmup:
            times.append(full)
            sampled.append(per_layer + head)
    full = sum(times) / len(times)
    step_s = sum(sampled) / len(sampled)   # what a step of this arm really ran: the bounded sample
    accepted = 1.0   # the oracle's pass emits at least the bonus token; drafts are not generated on this arm
    val = accepted / full
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val,
        "unit": "accepted tok/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": step_s * 1e3, "ms_per_pass_extrapolated": full * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": WORKLOAD, "replicas": 1, "batch": BATCH, "prefix": PREFIX, "gamma": GAMMA},
        "cpu_baseline": {"value": val, "unit": "accepted tok/s", "kind": "oracle", "cores": sample.threads,
                         "sample": "each step: 1 of 36 decoder layers + LM head at full widths, scaled to 36 layers; "
                                   "counts the bonus token only (1 token per pass)"},
        "e2e": {"value": val, "unit": "accepted tok/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def run_profile_pass(args):
    """For `ncu --profile-from-start off`: builds the int8 model only, warms up, then runs ONE eager verify
    pass between cudaProfilerStart/Stop.  Prints nothing that is a benchmark value."""
    from paper_2603_01399_b200 import binding, build
    build.build()
    torch.cuda.set_device(0)
    shape = synth.SHAPES["qwen3_8b"]
    if args.profile_layers:
        shape = synth.ModelShape("qwen3_8b_cut", args.profile_layers, shape.hidden, shape.n_q_heads, shape.n_kv_heads,
                                 shape.head_dim, shape.ffn, shape.vocab, shape.qk_norm, shape.rope_theta, shape.rms_eps)
    s_max = PREFIX + 16
    model = binding.Model.from_master(shape, master_getter(shape, 0, "cuda"), s_max, int8=True)
    kk, vv = synth.kv_prefix(shape, BATCH, s_max, seed=1, device="cuda")
    kv = binding.KVCache(shape, BATCH, s_max, k=kk, v=vv,
                         seq_len=torch.full((BATCH,), PREFIX, dtype=torch.int32, device="cuda"))
    buf = binding.VerifyBuffers(model, BATCH, GAMMA + 1, want_logits=False)
    buf.tokens.copy_(synth.uniform_tokens((BATCH, GAMMA + 1), shape.vocab, synth.sub_seed(2, "tokens")))
    for _ in range(3):
        binding.quasar_verify(model, kv, buf)
    torch.cuda.synchronize()
    torch.cuda.profiler.start()
    binding.quasar_verify(model, kv, buf)
    torch.cuda.synchronize()
    torch.cuda.profiler.stop()
    print(json.dumps({"profile_pass": "done", "layers": shape.n_layers, "status": int(buf.status[0])}))


def run_profile_linear(args):
    """For `ncu --profile-from-start off`: ONE quantised linear layer of a named Qwen3-8B shape at --rows rows
    (int8 weights; --a8: the W8A8 form) between cudaProfilerStart/Stop, after two warm-up calls."""
    from paper_2603_01399_b200 import binding, build
    build.build()
    torch.cuda.set_device(0)
    shapes = {"qkv": (4096, 6144), "o": (4096, 4096), "gateup": (4096, 24576), "down": (12288, 4096), "lm_head": (4096, 151936)}
    k, n = shapes[args.profile_linear]
    m = args.rows
    master = synth.normal_bf16((n, k), 0.02, seed=k + n, device="cuda")
    x = synth.normal_bf16((m, k), 1.0, seed=m, device="cuda")
    if args.a8:
        q, d = binding.quasar_quantize_weights_smoothed(master, None)
        call = lambda: binding.quasar_linear_w8a8(x, None, q, d)
    else:
        q, d = binding.quasar_quantize(master)
        ws = torch.zeros(binding.quasar_linear_workspace_bytes(m, n, k), dtype=torch.uint8, device="cuda")
        y = torch.empty((m, n), dtype=torch.bfloat16, device="cuda")
        call = lambda: binding.quasar_linear(x, q, d, workspace=ws, out=y)
    del master
    for _ in range(2):
        call()
    torch.cuda.synchronize()
    torch.cuda.profiler.start()
    call()
    torch.cuda.synchronize()
    torch.cuda.profiler.stop()
    print(json.dumps({"profile_linear": args.profile_linear, "rows": m, "a8": bool(args.a8), "weight_bytes": n * k}))


def run_profile_batch8(args):
    """For `ncu --profile-from-start off`: one eager pass of the batch-of-eight workload (prefixes U(512,4096),
    chains of 8 drafts, 72 block rows) on a model cut to --profile-layers layers."""
    from paper_2603_01399_b200 import binding, build
    build.build()
    torch.cuda.set_device(0)
    full = synth.SHAPES["qwen3_8b"]
    shape = synth.ModelShape("qwen3_8b_cut", args.profile_layers or 2, full.hidden, full.n_q_heads, full.n_kv_heads, full.head_dim,
                             full.ffn, full.vocab, full.qk_norm, full.rope_theta, full.rms_eps)
    absmax = (lambda kind, layer: synth.activation_absmax(shape, kind, layer, 0, "cuda")) if args.a8 else None
    model = binding.Model.from_master(shape, master_getter(shape, 0, "cuda"), 4096 + 16, int8=True, act_int8=bool(args.a8),
                                      get_act_absmax=absmax)
    rng = np.random.default_rng(4)
    prefix = [int(v) for v in rng.integers(512, 4097, 8)]
    kk, vv = synth.kv_prefix(shape, 8, 4096 + 16, seed=1, device="cuda")
    kv = binding.KVCache(shape, 8, 4096 + 16, k=kk, v=vv, seq_len=torch.tensor(prefix, dtype=torch.int32, device="cuda"))
    buf = binding.VerifyBuffers(model, 8, 9, want_logits=False)
    buf.tokens.copy_(synth.uniform_tokens((8, 9), shape.vocab, synth.sub_seed(2, "tokens")))
    for _ in range(2):
        binding.quasar_verify(model, kv, buf)
    torch.cuda.synchronize()
    torch.cuda.profiler.start()
    binding.quasar_verify(model, kv, buf)
    torch.cuda.synchronize()
    torch.cuda.profiler.stop()
    print(json.dumps({"profile_batch8": "done", "layers": shape.n_layers, "a8": bool(args.a8), "status": int(buf.status[0])}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--profile-pass", action="store_true",
                    help="run one eager verify pass inside cudaProfilerStart/Stop (for ncu), no timing")
    ap.add_argument("--profile-layers", type=int, default=0, help="with --profile-pass: cut the model to this many layers")
    ap.add_argument("--linear-sweep", action="store_true", help="time the quantised linear layer alone over shapes and row counts")
    ap.add_argument("--profile-linear", default="", help="one quantised linear layer of this Qwen3-8B shape inside cudaProfilerStart/Stop (for ncu)")
    ap.add_argument("--profile-batch8", action="store_true", help="one eager batch-of-eight pass inside cudaProfilerStart/Stop (for ncu)")
    ap.add_argument("--rows", type=int, default=72, help="with --profile-linear: activation rows")
    ap.add_argument("--a8", action="store_true", help="with --profile-linear / --profile-batch8: the W8A8 form")
    ap.add_argument("--headline-only", action="store_true", help="skip the side workloads (W8A8, linear sweep, 14B tree)")
    args = ap.parse_args()
    if args.profile_pass:
        return run_profile_pass(args)
    if args.profile_linear:
        return run_profile_linear(args)
    if args.profile_batch8:
        return run_profile_batch8(args)
    if args.linear_sweep:
        return run_linear_sweep(args)
    # --gpus N: N independent replicas (the pass has no exchange step), one process per GPU.  Launched
    # without a process launcher the replicas are started here; under torchrun the world size must agree.
    world_env = os.environ.get("WORLD_SIZE")
    if world_env is not None and int(world_env) != args.gpus:
        print(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world_env}", file=sys.stderr)
        sys.exit(2)
    if world_env is None and args.gpus > 1:
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
