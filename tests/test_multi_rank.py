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
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""
