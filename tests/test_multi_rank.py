"""The replica logic of bench.py with two ranks on CPU (gloo): the job's step time is the slowest rank's,
its throughput counts every rank's tokens, and only rank 0 of the reference arm does any work."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank = dist.get_rank()
    ms = bench.max_over_ranks(3.0 + rank, dist, "cpu")          # rank 1 is the slow one
    toks = bench.sum_over_ranks(2.0 + rank, dist, "cpu")        # every replica's accepted tokens count
    none = (bench.max_over_ranks(5.0, None, "cpu"), bench.sum_over_ranks(7.0, None, "cpu"))
    dist.barrier()
    print(json.dumps({"rank": rank, "ms": ms, "toks": toks, "none": none}), flush=True)
    dist.destroy_process_group()
""")


def test_two_rank_reductions_over_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29571", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-2000:]
    import json
    for o, _ in outs:
        rec = json.loads(o.strip().splitlines()[-1])
        assert rec["ms"] == 4.0 and rec["toks"] == 5.0 and rec["none"] == [5.0, 7.0]


def test_reference_arm_only_works_on_rank_zero():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""


def test_gpus_flag_starts_the_replicas_itself_and_checks_the_world_size():
    """`bench.py --gpus 2` without a launcher starts two replica processes (here: the reference arm, on CPU):
    exactly one JSON line comes back, from rank 0, with n_gpus 2; under a launcher a world size that
    disagrees with --gpus is refused."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=900)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
    assert rec["ms_per_step"] < rec["ms_per_pass_extrapolated"]
    bad = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--impl", "reference"],
                         env=dict(env, WORLD_SIZE="2", RANK="0", LOCAL_RANK="0"), capture_output=True, text=True, timeout=120)
    assert bad.returncode == 2 and "WORLD_SIZE" in bad.stderr
