"""Multi-process plumbing on CPU (gloo, world_size 2) and the benchmark's reference arm."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

from paper_2309_01507_b200 import dist, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    assert dist.init("gloo")
    dist.barrier()
    mx = dist.max_over_ranks(10.0 + rank)
    sm = dist.sum_over_ranks(1.0 + rank)
    dist.barrier()
    dist.shutdown()
    out.put((rank, mx, sm))


def test_barrier_and_max_over_ranks_gloo_world2():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29731, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 11.0, 3.0), (1, 11.0, 3.0)]


def test_single_process_helpers_are_noops():
    assert dist.env()[2] >= 1
    dist.barrier()
    assert dist.max_over_ranks(3.5) == 3.5


def test_partition_by_bytes_covers_and_balances():
    for wl in (workloads.transformer_base(), workloads.llama_7b()):
        numels = [t.numel for t in wl.tensors]
        for world in (1, 2, 4, 8):
            owned = dist.partition_by_bytes(numels, world)
            flat = sorted(i for o in owned for i in o)
            assert flat == list(range(len(numels)))
            loads = [sum(numels[i] for i in o) for o in owned]
            assert max(loads) <= sum(numels) / world + max(numels)


def test_reference_arm_prints_one_line_on_rank0_only():
    env = dict(os.environ, OMP_NUM_THREADS="4")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "single_matrix",
           "--steps", "1", "--warmup", "0"]
    out = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["value"] > 0 and rec["cpu_baseline"]["kind"] == "oracle"
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["unit"] == "Gparams/s"
    env1 = dict(env, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out1 = subprocess.run(cmd, env=env1, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out1.returncode == 0 and out1.stdout.strip() == ""
