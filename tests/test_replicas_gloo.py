"""The N>1 path on CPU: two gloo ranks exercise bench.py's rank plumbing (replicas only: no
data-path collective, per-rank seeds, max-over-ranks timing), and the reference arm under
torchrun prints exactly one line from rank 0."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    from paper_2409_15104_b200 import workloads
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = workloads.WORKLOADS["c3"]
    seed = bench.replica_seed(wl, rank)
    times = bench.max_over_ranks([10.0 + 5 * rank, 3.0 - rank], dist, "cpu")
    dist.barrier()
    out.put((rank, seed, times, bench.whole_job_tflops(1e12, world, times[0])))
    dist.destroy_process_group()


def test_two_ranks_take_max_time_and_own_seeds():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, t0, f0), (r1, s1, t1, f1) = res
    assert s0 != s1
    assert t0 == t1 == [15.0, 3.0]                 # slowest rank decides
    assert f0 == f1 == 2 * 1e12 / 15e-3 / 1e12     # both replicas' work over that time


def test_reference_arm_under_torchrun_prints_one_line_from_rank_zero():
    port = 31500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port),
           os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
           "--reference-seconds", "1"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"]
    assert line["value"] > 0 and line["unit"] == "TFLOP/s"
