"""The N > 1 path on CPU (gloo, world size 2): replicas share nothing on the data path, so what
several ranks add is the timing reduction (maximum over ranks), the whole-job throughput formula,
and the rule that only rank 0 reports.  Also the reference arm launched the way the driver launches
it for N = 2: rank 0 prints one JSON line, the other rank exits 0 without work."""
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
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [10.0 + 5.0 * rank, 3.0 - rank]            # rank 1 is slower on the first, faster on the second
        got = bench.max_over_ranks(dist, mine, "cpu")
        dist.barrier()
        out.put((rank, got, bench.whole_job_throughput(world, 8, 100, got[0])))
    finally:
        dist.destroy_process_group()


def test_timing_reduction_and_throughput_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, thr in res:
        assert got == [15.0, 3.0]                          # maximum over ranks, same on every rank
        assert abs(thr - 2 * 8 * 100 / 15.0e-3) < 1e-6    # units of both ranks over the slowest rank's time
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(None, [1.5, 2], "cpu") == [1.5, 2.0]


def test_reference_arm_under_torchrun_with_two_ranks():
    port = 31500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "1", "--warmup", "0"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                  # rank 0 alone reports
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["unit"] == "tokens/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
