"""The N > 1 path of bench.py on CPU: two gloo ranks exercise the launcher
environment parsing, the per-rank batch shards (no data-path collective: FPROP
has no exchange step; the filter gradient's sum over ranks is the one exception), the max-over-ranks timing reduction and the whole-job
throughput; and the reference arm under a 2-rank launcher prints exactly one line."""
import json
import os
import subprocess
import sys

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import bench
    from paper_1501_06633_b200 import workloads as wl
    assert bench.rank_env() == (rank, rank, world)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.WORKLOADS["tiny3x3"]
    inp, filt = bench.shard_inputs(w, rank)
    # each rank "measures" a different time; everyone must end up with the slowest
    ms_total, e2e_ms = bench.max_over_ranks([10.0 + rank, 100.0 - rank], "cpu", world)
    import torch
    grad = bench.sum_gradient_over_ranks(torch.full((5,), float(rank + 1)), world)
    assert bool((grad == 3.0).all())               # 1 + 2: every rank holds the summed gradient
    dist.barrier()
    q.put((rank, float(inp.sum()), float(filt.sum()), ms_total, e2e_ms))
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_and_reduce():
    world, port = 2, 29500 + (os.getpid() % 2000)
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, in0, f0, ms0, e0), (_, in1, f1, ms1, e1) = res
    assert in0 != in1 and f0 != f1                 # independent shards of the same recipe
    assert ms0 == ms1 == 11.0 and e0 == e1 == 100.0  # max over ranks, on every rank
    import bench
    assert np.isclose(bench.whole_job_tflops(2e12, 2, 1000.0), 4.0)


def test_reference_arm_under_a_two_rank_launcher_prints_one_line():
    env = dict(os.environ, OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(31000 + os.getpid() % 2000),
           os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--workload", "tiny3x3"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["e2e"]["h2d_bytes_per_step"] == 0
