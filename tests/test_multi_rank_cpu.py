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


# ---- a decode step's keys spread over two ranks: range cutting, all-gather layout, merge ---------------

def _keysplit_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import numpy as np
    import oracle
    from paper_2604_07394_b200 import keysplit
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(77)                    # same inputs on every rank
        Hq, Hkv, D, S, W = 4, 2, 8, 3, 5
        lens, modes = [40, 9, 23], [1, 0, 0]               # one dense request, one sparse that keeps all, one truly sparse
        B, G = len(lens), Hq // Hkv
        ranges = keysplit.key_ranges(lens, world, align=4)
        q = [oracle.f64_to_bits(rng.standard_normal((Hq, D))) for _ in lens]
        K = [oracle.f64_to_bits(rng.standard_normal((n, Hkv, D))) for n in lens]
        V = [oracle.f64_to_bits(rng.standard_normal((n, Hkv, D))) for n in lens]
        # this rank's piece, by the oracle, with the rule the library states: a dense walk takes the rows of its
        # range, a sparse request goes whole to the range that holds its newest position
        po = np.zeros((B, Hq, D)); pml = np.zeros((B, Hq, 2)); pml[..., 0] = -np.inf
        for b, n in enumerate(lens):
            kb, ke = int(ranges[rank, b, 0]), int(ranges[rank, b, 1])
            kept = oracle.kept(modes[b], n - 1, S, W)
            if modes[b] == 1 or n <= S + W:
                idx = kept[(kept >= kb) & (kept < ke)]
            else:
                idx = kept if kb <= n - 1 < ke else kept[:0]
            for h in range(Hq):
                if len(idx) == 0:
                    continue
                o, _, m, l = oracle.attend(q[b][h], K[b][:, h // G], V[b][:, h // G], idx, 0.3)
                po[b, h], pml[b, h] = o, (m, l)            # normalised output, natural-log maximum, sum
        got_o, got_ml = keysplit.all_gather_pieces(dist, torch.from_numpy(po), torch.from_numpy(pml))
        assert tuple(got_o.shape) == (world, B, Hq, D) and tuple(got_ml.shape) == (world, B, Hq, 2)
        assert torch.equal(got_o[rank], torch.from_numpy(po))          # rank-major layout
        worst = 0.0
        for b, n in enumerate(lens):
            ref = oracle.decode(modes[b], q[b], K[b], V[b], n, S, W, 0.3)
            for h in range(Hq):
                m, l, o = 0.0, 0.0, None
                for r in range(world):
                    mp, lp = float(got_ml[r, b, h, 0]), float(got_ml[r, b, h, 1])
                    if lp == 0.0:
                        continue
                    op = got_o[r, b, h].numpy()
                    m, l, o = (mp, lp, op) if o is None else oracle.merge(m, l, o, mp, lp, op)
                worst = max(worst, float(np.abs(o - ref[h]).max()))
        out.put((rank, worst, ranges.tolist()))
    finally:
        dist.destroy_process_group()


def test_key_ranges_gather_and_merge_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 33500 + os.getpid() % 2000
    procs = [ctx.Process(target=_keysplit_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][2] == res[1][2]                            # both ranks cut the same ranges
    ranges = res[0][2]
    assert [ranges[0][b][0] for b in range(3)] == [0, 0, 0] and [ranges[1][b][1] for b in range(3)] == [40, 9, 23]
    assert all(ranges[0][b][1] == ranges[1][b][0] and ranges[0][b][1] % 4 == 0 for b in range(3))
    for rank, worst, _ in res:
        assert worst < 1e-12                                 # merged pieces = the whole step, on every rank
