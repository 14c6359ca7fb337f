#!/usr/bin/env python
"""Benchmark of the routed hybrid attention hot path on B200.

Default arm (`--impl ours`): one *step* is one decode step of the whole routed stack
(per layer: KV append, mixed FA/SA split-K decode, combine) for the batched long-context decode
workload (32 layers, 32/8 heads, batch 8, 64K-token caches, half of each request's layers
sparse).  The line also carries the prefill measurement of the 32K-token workload as a
sub-object.  `--impl reference` times the fp64 CPU oracle on a bounded sample of the same
workload.  One JSON line on stdout (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2604_07394_b200 import synth  # noqa: E402

D = 128


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def traffic_note(kernel):
    """DRAM bytes per algorithmic byte of `kernel`, from the committed ncu summary (or None)."""
    p = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(p):
        return None
    with open(p) as f:
        return json.load(f).get(kernel)


# ---- multi-rank bookkeeping (replicas: no data-path collective, only the timing reduction) -----

def max_over_ranks(dist, values, device):
    """Element-wise maximum of per-rank timings over all ranks (identity without a process group)."""
    if dist is None:
        return [float(v) for v in values]
    tt = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return [float(v) for v in tt]


def whole_job_throughput(world, units_per_rank_step, steps, ms_max):
    """Units all ranks processed per second, over the slowest rank's time (weak scaling)."""
    return world * units_per_rank_step * steps / (ms_max / 1e3)


# ---- clocks ------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 6:
                    continue
                try:
                    sm.append(float(parts[0])); mx.append(float(parts[1]))
                except ValueError:
                    continue
                for nm, val in zip(names, parts[2:6]):
                    if val.lower().startswith("active"):
                        reasons.add(nm)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        hi = [s for s in sm if s >= 0.5 * max(sm)]          # samples under load
        return {"sm_mhz": float(np.median(hi)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


# ---- decode workload -----------------------------------------------------------------------------

class DecodeBench:
    def __init__(self, flux, w, dev, total_steps, host_mirrors=True):
        self.flux, self.w, self.dev = flux, w, dev
        B, L, Hq, Hkv = w.batch, w.n_layers, w.n_q_heads, w.n_kv_heads
        self.mask = synth.layer_masks(w)
        self.ctx0 = synth.context_lengths(w)
        self.total_steps = total_steps
        max_ctx = int(self.ctx0.max()) + total_steps + 1
        cfg = flux.make_config(L, Hq, Hkv, w.sink, w.window, B, max_ctx, kv_layout=flux.FLUX_KV_COMPACT_SA)
        self.plan = flux.Plan(cfg, dev)
        self.plan.flux_router_apply(logits=synth.masks_to_logits(self.mask, w.seed))
        assert np.array_equal(self.plan.mask.cpu().numpy(), self.mask)
        self.kc, self.vc = [], []
        nbytes = 0
        for l in range(L):
            kl, vl = [], []
            for b in range(B):
                rows = (w.sink + w.window) if self.mask[b, l] == 0 else int(self.ctx0[b]) + total_steps + 1
                k = torch.empty((rows, Hkv, D), dtype=torch.bfloat16, device=dev)
                v = torch.empty_like(k)
                synth.fill_normal_bf16_(k, w.seed, synth.stream_id("k", l, b))
                synth.fill_normal_bf16_(v, w.seed, synth.stream_id("v", l, b))
                kl.append(k); vl.append(v)
                nbytes += 2 * k.numel() * 2
            self.kc.append(kl); self.vc.append(vl)
        self.cache_bytes = nbytes
        self.ktab = [flux.pointer_table(self.kc[l], dev) for l in range(L)]
        self.vtab = [flux.pointer_table(self.vc[l], dev) for l in range(L)]
        self.q = synth.normal_bf16((L, B, Hq, D), w.seed, synth.stream_id("qdec"), dev)
        self.kn = synth.normal_bf16((L, B, Hkv, D), w.seed, synth.stream_id("kdec"), dev)
        self.vn = synth.normal_bf16((L, B, Hkv, D), w.seed, synth.stream_id("vdec"), dev)
        self.out = torch.empty_like(self.q)
        steps = np.arange(total_steps + 1, dtype=np.int32)[:, None]
        self.ctx_host = self.ctx0[None, :].astype(np.int32) + steps + 1      # [T+1][B] context incl. new token
        self.ctx = torch.from_numpy(self.ctx_host).to(dev)
        self.pos = self.ctx - 1
        if host_mirrors:            # for the end-to-end arm
            self.q_h = self.q.cpu().pin_memory(); self.kn_h = self.kn.cpu().pin_memory()
            self.vn_h = self.vn.cpu().pin_memory(); self.out_h = torch.empty_like(self.q_h).pin_memory()

    def step(self, t):
        p, w = self.plan, self.w
        for l in range(w.n_layers):      # append + attend of a layer in one launch, then the combine pass
            p.flux_attn_decode_step(l, w.batch, self.q[l], self.kn[l], self.vn[l], self.ktab[l], self.vtab[l],
                                    self.ctx[t], self.out[l])

    def capture_step(self, t_next):
        """One decode step (all layers) as a CUDA graph.  The step's positions live in two device
        vectors the graph itself advances, so every replay is the next step."""
        p, w = self.plan, self.w
        self.ctx_cur = self.ctx[t_next].clone()
        self.pos_cur = self.pos[t_next].clone()
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            for l in range(w.n_layers):
                p.flux_attn_decode_step(l, w.batch, self.q[l], self.kn[l], self.vn[l], self.ktab[l], self.vtab[l],
                                        self.ctx_cur, self.out[l])
            self.ctx_cur += 1
            self.pos_cur += 1
        torch.cuda.synchronize()

    def step_graph(self):
        self.graph.replay()

    def step_host(self, t):
        p, w = self.plan, self.w
        for l in range(w.n_layers):
            p.flux_attn_decode_host(l, w.batch, self.q_h[l], self.kn_h[l], self.vn_h[l], self.ktab[l],
                                    self.vtab[l], self.pos[t], self.ctx[t], self.out_h[l])

    def kept_rows(self, t):
        """[B][L] KV rows the method must read at step t."""
        n = self.ctx_host[t][:, None].astype(np.int64)
        sw = self.w.sink + self.w.window
        return np.where(self.mask == 1, n, np.minimum(n, sw))

    def bytes_step(self, t):
        return int(self.kept_rows(t).sum()) * 2 * self.w.n_kv_heads * D * 2

    def h2d_bytes(self):
        w = self.w
        return w.n_layers * w.batch * (w.n_q_heads + 2 * w.n_kv_heads) * D * 2

    def d2h_bytes(self):
        w = self.w
        return w.n_layers * w.batch * w.n_q_heads * D * 2


def logical_cache(cache_rows_cpu, n, S, W, compact):
    """Position-indexed [n][Hkv][D] view of a cache copy (evicted rows zero)."""
    import oracle
    if not compact:
        return cache_rows_cpu[:n]
    out = torch.zeros((n,) + tuple(cache_rows_cpu.shape[1:]), dtype=cache_rows_cpu.dtype)
    keep = oracle.retained(n, S, W)
    slots = np.array([oracle.compact_slot(int(j), S, W) for j in keep])
    out[torch.from_numpy(keep)] = cache_rows_cpu[torch.from_numpy(slots)]
    return out


def cpu_baseline_decode(db: DecodeBench):
    """Oracle on a bounded sample of step 0: every request, its first FA and first SA layer, all
    heads; checks the GPU output on those rows and extrapolates the oracle's tokens/s."""
    import oracle
    from tests._util import compare     # the parity tests' comparison rule
    w = db.w
    t = 0
    db.step(t)
    torch.cuda.synchronize()
    scale = 1.0 / np.sqrt(D)
    t_mode = {0: [], 1: []}
    worst = 0.0
    threads = os.cpu_count() or 1
    sample = [(b, mode, int(l)) for b in range(w.batch) for mode in (1, 0)
              for l in np.nonzero(db.mask[b] == mode)[0][:3]]
    for b, mode, l in sample:
        n = int(db.ctx_host[t][b])
        compact = mode == 0
        k = logical_cache(db.kc[l][b].cpu(), n, w.sink, w.window, compact)
        v = logical_cache(db.vc[l][b].cpu(), n, w.sink, w.window, compact)
        qb, kb, vb = oracle.to_bits(db.q[l, b].cpu()), oracle.to_bits(k), oracle.to_bits(v)
        t0 = time.perf_counter()
        ref = oracle.decode(mode, qb, kb, vb, n, w.sink, w.window, scale)
        t_mode[mode].append(time.perf_counter() - t0)
        _, rel, _ = compare(db.out[l, b], ref, "bench parity b=%d layer=%d mode=%d" % (b, l, mode))
        worst = max(worst, rel)
    t_fa = float(np.mean(t_mode[1])) if t_mode[1] else 0.0
    t_sa = float(np.mean(t_mode[0])) if t_mode[0] else 0.0
    n_fa = int((db.mask == 1).sum()); n_sa = int((db.mask == 0).sum())
    step_s = n_fa * t_fa + n_sa * t_sa
    return {"value": w.batch / step_s, "unit": "tokens/s", "cores": threads, "kind": "oracle",
            "sample": "step 0, all %d requests, first 3 FA and first 3 SA layers of each, all %d heads "
                      "(%d (request,layer) rows sets, %.1f s of oracle time); extrapolated to the full "
                      "step by FA/SA layer counts" % (w.batch, w.n_q_heads, len(t_mode[0]) + len(t_mode[1]),
                                                      sum(t_mode[0]) + sum(t_mode[1])),
            "parity_max_row_rel": worst}


def timed_replays(db, steps):
    """`steps` graph replays bracketed by CUDA events on the current stream -> milliseconds."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        db.step_graph()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def kernel_roofline(db, flux, t, steps, peaks, kernel_name):
    """The dominant decode kernel, event-bracketed launch by launch on `steps` steps issued call by call."""
    w = db.w
    db.plan.flux_profile_enable(steps * w.n_layers + 8)
    for i in range(steps):
        db.step(t + i)
    torch.cuda.synchronize()
    kms, kcnt = db.plan.flux_profile_read(flux.FLUX_KERNEL_DECODE)
    db.plan.flux_profile_enable(0)
    by = sum(db.bytes_step(t + i) for i in range(steps)) / max(kcnt, 1)
    ms = kms / max(kcnt, 1)
    ach = by / (ms * 1e-3) / 1e9
    return {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
            "peak_source": peaks["source"] + " (copy bandwidth)", "kernel": kernel_name, "launches_timed": int(kcnt),
            "avg_launch_ms": ms, "algorithmic_bytes_per_launch": by}


def decode_kernel_name(flux, plan_choice, batch):
    single = plan_choice != "two_launch" and batch <= 32
    return ("decode_fused_kernel (split-K decode and merge in one launch per layer)" if single else
            "decode_kernel (mixed FA/SA split-K decode, one launch per layer)")


def secondary_decode_block(flux, dev, peaks, name, steps, warmup, args):
    """Another decode workload, device-resident: graph replays of the whole step, required bytes / time
    against the measured HBM copy bandwidth, and its dominant kernel launch by launch."""
    import dataclasses
    w = synth.WORKLOADS[name]
    if w.prompt_len:                       # the decode phase of a prefill + decode workload: the cache is drawn directly
        w = dataclasses.replace(w, prompt_len=0)
    roof_steps = 5
    db = DecodeBench(flux, w, dev, 1 + 2 * warmup + steps + roof_steps + 2, host_mirrors=False)
    db.plan.flux_debug_decode_kernel({"auto": flux.FLUX_DECODE_AUTO, "two_launch": flux.FLUX_DECODE_TWO_LAUNCH,
                                      "single_launch": flux.FLUX_DECODE_SINGLE_LAUNCH}[args.decode_kernel])
    db.plan.flux_plan_set_launch_overlap(not args.no_launch_overlap)
    t = 0
    for _ in range(warmup):
        db.step(t); t += 1
    n0 = db.plan.flux_launch_count()
    db.capture_step(t)
    per_step = db.plan.flux_launch_count() - n0
    timed_replays(db, warmup); t += warmup
    t_first = t
    ms = timed_replays(db, steps); t += steps
    by = sum(db.bytes_step(i) for i in range(t_first, t_first + steps))
    roof = kernel_roofline(db, flux, t, roof_steps, peaks, decode_kernel_name(flux, args.decode_kernel, w.batch))
    assert db.plan.flux_plan_status() == 0
    gbs = by / (ms * 1e-3) / 1e9
    if per_step == w.n_layers:     # one launch per layer and nothing else in the step: the graph region times the kernel itself
        roof.update({"event_bracketed": {"avg_launch_ms": roof["avg_launch_ms"], "gbs": roof["achieved"]},
                     "achieved": gbs, "frac": gbs / peaks["hbm_gbs"], "launches_timed": steps * w.n_layers,
                     "avg_launch_ms": ms / (steps * w.n_layers), "algorithmic_bytes_per_launch": by / (steps * w.n_layers),
                     "timing": "timed region of the graph replays / launches (dense and sparse layers averaged together)"})
    res = {"workload": workload_config(w, db.mask, db.ctx0)["workload"], "tokens_per_s": w.batch * steps / (ms * 1e-3),
           "ms_per_step": ms / steps, "steps": steps, "required_bytes_per_step": by / steps,
           "step_level_gbs": gbs, "step_level_frac_of_hbm_peak": gbs / peaks["hbm_gbs"],
           "gpu_launches_per_step": int(per_step), "omega_msr": float((db.mask == 0).mean()), "roofline": roof}
    del db
    torch.cuda.empty_cache()
    return res


# ---- Layer Router front end (Sec. 3.1): latency per layer -------------------------------------------

def router_frontend_block(flux, dev, peaks, warmup, enc_dim=1024, head_hidden=256):
    """x_Q segments -> logits for every layer of the cfg2 stack, then the hard decision; the paper
    quotes 0.20 ms per layer for its router (Sec. 4.3).  Widths are this benchmark's choice (the
    paper gives none).  Timed with CUDA events over `reps` passes of all layers."""
    w = synth.WORKLOADS["cfg2"]
    L, Hq, Hkv = w.n_layers, w.n_q_heads, w.n_kv_heads
    F = 2 * Hq * D
    plan = flux.Plan(flux.make_config(L, Hq, Hkv, w.sink, w.window, 1, 4096), dev)
    q = synth.normal_bf16((4096, Hq, D), w.seed, synth.stream_id("q"), dev)
    ws = [synth.router_weights(w.seed, l, F, enc_dim, head_hidden, dev) for l in range(L)]
    logits = torch.zeros((1, L, 2), dtype=torch.float32, device=dev)
    first, last = q[:100], q[-100:]

    def one_pass():
        for l in range(L):
            plan.flux_router_forward(ws[l], first, last, logits[0, l])
        return plan.flux_router_apply(logits=logits)

    for _ in range(max(3, warmup)):
        one_pass()
    torch.cuda.synchronize()
    reps = 20
    n0 = plan.flux_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        mask = one_pass()
    e1.record()
    torch.cuda.synchronize()
    ms_eager = e0.elapsed_time(e1) / reps
    launches = int(plan.flux_launch_count() - n0) // reps
    # the same pass as one CUDA graph: the device's own time per layer, without the host's call overhead
    ms = ms_eager
    stepping = "issued call by call (the host's call overhead is inside the number)"
    try:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            one_pass()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        stepping = "one CUDA graph per pass over all layers, replayed %d times" % reps
    except Exception as e:          # report, never hide
        stepping += "; graph capture failed: %r" % (e,)
    assert plan.flux_plan_status() == 0
    bytes_layer = 2 * (F * enc_dim + enc_dim * enc_dim + enc_dim * head_hidden + 2 * head_hidden) + 2 * 200 * Hq * D
    return {"workload": "cfg2 stack: 32 layers, x_Q of 32 heads x 128, first 100 + last 100 tokens pooled; "
                        "encoder width %d, head hidden %d (benchmark's choice)" % (enc_dim, head_hidden),
            "us_per_layer": ms * 1e3 / L, "ms_all_layers_and_decision": ms, "stepping": stepping,
            "us_per_layer_call_by_call": ms_eager * 1e3 / L,
            "algorithmic_bytes_per_layer": bytes_layer,
            "gbs": bytes_layer * L / (ms * 1e-3) / 1e9, "hbm_peak_gbs": peaks["hbm_gbs"],
            "bound": "dependency latency (%d launch per layer, five dependent stages handed over through L2, %.1f MB of weights per layer)"
                     % ((launches - 1) // L, bytes_layer / 1e6),
            "hbm_floor_us_per_layer": bytes_layer / (peaks["hbm_gbs"] * 1e9) * 1e6,
            "gpu_launches": launches,
            "omega_msr_random_weights": float((mask == 0).float().mean()),
            "paper_router_ms_per_layer": 0.20}


# ---- prefill workload ------------------------------------------------------------------------------

def prefill_block(flux, dev, peaks, warmup):
    w = synth.WORKLOADS["cfg2"]
    N, L, Hq, Hkv, S, W = w.prompt_len, w.n_layers, w.n_q_heads, w.n_kv_heads, w.sink, w.window
    mask = synth.layer_masks(w)
    cfg = flux.make_config(L, Hq, Hkv, S, W, 1, N)
    plan = flux.Plan(cfg, dev)
    plan.flux_router_apply(mask=mask)
    q = synth.normal_bf16((N, Hq, D), w.seed, synth.stream_id("q"), dev)
    k = synth.normal_bf16((N, Hkv, D), w.seed, synth.stream_id("k"), dev)
    v = synth.normal_bf16((N, Hkv, D), w.seed, synth.stream_id("v"), dev)
    out = torch.empty_like(q)
    fa_layers = [l for l in range(L) if mask[0, l] == 1]
    sa_layers = [l for l in range(L) if mask[0, l] == 0]
    for l in (fa_layers[:1] + sa_layers[:1]) * max(1, warmup):
        plan.flux_attn_prefill(l, 0, q, k, v, 0, out)
    torch.cuda.synchronize()

    def timed(layers):
        plan.flux_profile_enable(len(layers) + 1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for l in layers:
            plan.flux_attn_prefill(l, 0, q, k, v, 0, out)
        e1.record()
        torch.cuda.synchronize()
        kms, cnt = plan.flux_profile_read(flux.FLUX_KERNEL_PREFILL)
        plan.flux_profile_enable(0)
        return e0.elapsed_time(e1), kms, cnt

    res = {}
    i = np.arange(N, dtype=np.int64)
    pairs_fa = int((i + 1).sum())
    pairs_sa = int(np.minimum(i + 1, S + W).sum())
    flop_fa, flop_sa = 4 * Hq * D * pairs_fa, 4 * Hq * D * pairs_sa
    ms_fa = ms_sa = None
    if fa_layers:
        _, kms, cnt = timed(fa_layers)
        ms_fa = kms / cnt
    if sa_layers:
        _, kms, cnt = timed(sa_layers)
        ms_sa = kms / cnt
    wall_ms, kms_all, cnt_all = timed(list(range(L)))
    total_flop = len(fa_layers) * flop_fa + len(sa_layers) * flop_sa
    res = {
        "workload": "cfg2: 32 layers, 32/8 heads, d128, batch 1, prefill 32768 tokens, sink 128 + window 2048, "
                    "Bernoulli(0.5) layer mask from seed (%d FA / %d SA)" % (len(fa_layers), len(sa_layers)),
        "ms_per_layer_mix": wall_ms, "ms_fa_layer": ms_fa, "ms_sa_layer": ms_sa,
        "tflops_fa": None if ms_fa is None else flop_fa / ms_fa / 1e9,
        "tflops_sa": None if ms_sa is None else flop_sa / ms_sa / 1e9,
        "tflops_mix": total_flop / wall_ms / 1e9,
        "gpu_launches": cnt_all,
    }
    # the same sparse pattern at block granularity (64-position blocks) through the block-mask entry point
    nb = N // 64
    qb = np.arange(nb)[:, None]; kb = np.arange(nb)[None, :]
    bm = ((kb <= qb) & ((kb < -(-S // 64)) | (kb > qb - -(-W // 64)))).astype(np.uint8)
    bm_dev = torch.from_numpy(bm).to(dev)
    for _ in range(max(1, warmup)):
        plan.flux_attn_prefill_blocks(q, k, v, 0, bm_dev, out)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        plan.flux_attn_prefill_blocks(q, k, v, 0, bm_dev, out)
    e1.record()
    torch.cuda.synchronize()
    ms_blk = e0.elapsed_time(e1) / 5
    off = bm.sum(axis=1).astype(np.int64) - 1                     # kept blocks below the diagonal, per query block
    pairs_blk = int((off * 64 * 64).sum() + nb * (64 * 65 // 2))  # + the causal half of each diagonal block
    res["block_mask_sa"] = {"kernel": "prefill_tc_kernel in block-mask mode (64 x 64 blocks inside 128 x 128 tiles)", "pattern":
                            "streaming at block granularity: %d sink + %d local blocks" % (-(-S // 64), -(-W // 64)),
                            "ms_layer": ms_blk, "tflops": 4 * Hq * D * pairs_blk / ms_blk / 1e9}
    if ms_fa is not None:
        # the same FA launch timed alone: one launch after the GPU has been idle for a while, which is how the burst
        # peak of the roofline's denominator was taken (the loop above runs under the power cap, like the sustained one)
        alone = []
        for _ in range(3):
            time.sleep(1.5)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            plan.flux_attn_prefill(fa_layers[0], 0, q, k, v, 0, out)
            e1.record()
            torch.cuda.synchronize()
            alone.append(e0.elapsed_time(e1))
        ms_alone = sorted(alone)[1]
        res["fa_layer_timed_alone"] = {"ms": ms_alone, "tflops": flop_fa / ms_alone / 1e9,
                                       "frac_of_burst_peak": flop_fa / ms_alone / 1e9 / peaks["bf16_tflops"],
                                       "how": "one launch after 1.5 s of idle, event-timed, median of 3 (%s ms)"
                                              % ", ".join("%.3f" % x for x in alone)}
        ach = flop_fa / ms_fa / 1e9
        res["roofline"] = {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops_sustained"],
                           "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops_sustained"],
                           "frac_of_burst_peak": ach / peaks["bf16_tflops"],
                           "peak_source": peaks["source"] + " (sustained cuBLAS bf16)",
                           "kernel": "FA prefill layer",
                           "traffic": (traffic_note("prefill_fa") or {}).get("dram_bytes_per_launch"),
                           "traffic_source": (traffic_note("prefill_fa") or {}).get("source")}
    plan.close()
    return res


def prefill_128k_block(flux, dev, peaks, warmup):
    """One FA and one SA layer of the 128K-token prefill (28 query / 4 KV heads: an odd group of 7, which
    leaves one head per KV group to the two-row-tiles item shape), each timed alone."""
    w = synth.WORKLOADS["cfg4"]
    N, Hq, Hkv, S, W = w.prompt_len, w.n_q_heads, w.n_kv_heads, w.sink, w.window
    plan = flux.Plan(flux.make_config(2, Hq, Hkv, S, W, 1, N), dev)
    plan.flux_router_apply(mask=np.array([[1, 0]], dtype=np.uint8))
    q = synth.normal_bf16((N, Hq, D), w.seed, synth.stream_id("q"), dev)
    k = synth.normal_bf16((N, Hkv, D), w.seed, synth.stream_id("k"), dev)
    v = synth.normal_bf16((N, Hkv, D), w.seed, synth.stream_id("v"), dev)
    out = torch.empty_like(q)
    i = np.arange(N, dtype=np.int64)
    flop = {0: 4 * Hq * D * int((i + 1).sum()), 1: 4 * Hq * D * int(np.minimum(i + 1, S + W).sum())}
    ms = {}
    for layer, reps in ((1, 3), (0, 2)):
        plan.flux_attn_prefill(layer, 0, q, k, v, 0, out)        # warm-up (an SA layer first: 8 ms)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            plan.flux_attn_prefill(layer, 0, q, k, v, 0, out)
        e1.record()
        torch.cuda.synchronize()
        ms[layer] = e0.elapsed_time(e1) / reps
    assert plan.flux_plan_status() == 0
    plan.close()
    del q, k, v, out
    torch.cuda.empty_cache()
    tf_fa, tf_sa = flop[0] / ms[0] / 1e9, flop[1] / ms[1] / 1e9
    n_fa, n_sa = int((synth.layer_masks(w) == 1).sum()), int((synth.layer_masks(w) == 0).sum())
    return {"workload": "cfg4 prefill: 28/4 heads, d128, batch 1, 131072 tokens in one call per layer, sink 128 + window 4096",
            "ms_fa_layer": ms[0], "ms_sa_layer": ms[1], "tflops_fa": tf_fa, "tflops_sa": tf_sa,
            "ms_whole_stack_from_layer_times": n_fa * ms[0] + n_sa * ms[1], "layers": "%d FA + %d SA" % (n_fa, n_sa),
            "roofline": {"bound": "tensor", "achieved": tf_fa, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                         "frac": tf_fa / peaks["bf16_tflops_sustained"], "frac_of_burst_peak": tf_fa / peaks["bf16_tflops"],
                         "peak_source": peaks["source"] + " (sustained cuBLAS bf16)", "kernel": "FA prefill layer (0.1 s per launch)",
                         "traffic": None}}


# ---- the paper's two ratios, re-measured on this GPU (context, not the headline) -----------------

def paper_ratio_block(flux, dev, warmup):
    """Decode-kernel and prefill speed of the routed stack against the all-FA stack at the paper's
    headline length (256K tokens, batch 1, Llama-3-8B attention shapes, sink 128 + window 2048,
    half of the layers sparse), to set beside the paper's 'approaching 2.0x' (decode kernels) and
    'up to 2.8x' (prefill, end to end, another sparse pattern); Sec. 4.3."""
    import dataclasses
    n, S, W, L = 262144, 128, 2048, 32
    base = dataclasses.replace(synth.WORKLOADS["cfg3"], batch=1, ctx_lo=n, ctx_hi=n, sink=S, window=W)
    res = {"context": n, "sink": S, "window": W}
    steps = 20
    times = {}
    for name, w in (("dense", dataclasses.replace(base, mask_rule="fixed", mask_arg=tuple([1] * L))),
                    ("routed", base)):
        db = DecodeBench(flux, w, dev, steps + warmup + 4, host_mirrors=False)
        db.plan.flux_plan_set_launch_overlap(True)
        t = 0
        db.step(t); t += 1
        db.capture_step(t)
        for _ in range(warmup):
            db.step_graph(); t += 1
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            db.step_graph(); t += 1
        e1.record()
        torch.cuda.synchronize()
        assert db.plan.flux_plan_status() == 0
        times[name] = e0.elapsed_time(e1) / steps
        omega = float((db.mask == 0).mean())
        del db
        torch.cuda.empty_cache()
    model = 1.0 / ((1 - omega) + omega * (S + W) / n)
    res["decode"] = {"dense_ms_per_step": times["dense"], "routed_ms_per_step": times["routed"],
                     "speedup": times["dense"] / times["routed"], "omega_msr": omega, "byte_model_speedup": model,
                     "paper": "decode attention kernels: approaching 2.0x at 256K (one A800 80GB, bf16, batch 1)"}
    # prefill in chunks of 16384 queries (Appendix D.3), one FA and one SA layer
    Hq, Hkv, C = base.n_q_heads, base.n_kv_heads, 16384
    plan = flux.Plan(flux.make_config(2, Hq, Hkv, S, W, 1, n), dev)
    plan.flux_router_apply(mask=np.array([[1, 0]], dtype=np.uint8))
    q = synth.normal_bf16((n, Hq, D), base.seed, synth.stream_id("q"), dev)
    k = synth.normal_bf16((n, Hkv, D), base.seed, synth.stream_id("k"), dev)
    v = synth.normal_bf16((n, Hkv, D), base.seed, synth.stream_id("v"), dev)
    out = torch.empty((C, Hq, D), dtype=torch.bfloat16, device=dev)
    ms = {}
    for layer in (1, 0):
        for a in range(0, min(n, 2 * C), C):          # warm-up on the first chunks
            plan.flux_attn_prefill(layer, 0, q[a:a + C], k[:a + C], v[:a + C], a, out)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for a in range(0, n, C):
            plan.flux_attn_prefill(layer, 0, q[a:a + C], k[:a + C], v[:a + C], a, out)
        e1.record()
        torch.cuda.synchronize()
        ms[layer] = e0.elapsed_time(e1)
    assert plan.flux_plan_status() == 0
    plan.close()
    i = np.arange(n, dtype=np.int64)
    flop_fa = 4 * Hq * D * int((i + 1).sum())
    flop_sa = 4 * Hq * D * int(np.minimum(i + 1, S + W).sum())
    res["prefill"] = {"chunk": C, "fa_layer_ms": ms[0], "sa_layer_ms": ms[1], "tflops_fa": flop_fa / ms[0] / 1e9,
                      "tflops_sa": flop_sa / ms[1] / 1e9,
                      "attention_speedup_half_layers_sparse": 2 * ms[0] / (ms[0] + ms[1]),
                      "paper": "prefill: up to 2.8x at 256K, end to end, Full + Triangle sparse mode (hardware not "
                               "stated beside the figure; latency set-up names one A800 80GB)"}
    return res


# ---- head-level vs layer-level sparsity at the same KV byte budget (Sec. 2.3, Appendix C.3) ----------

def head_level_block(flux, dev, peaks, warmup, n=262144, reps=30):
    """The paper's efficiency argument re-measured on this GPU: batch 1, Llama-3-8B attention shapes,
    sink 128 + window 2048, half of the KV bytes sparse.  Layer-level: half of the layers sparse
    (one dense layer call + one sparse layer call stand for a pair of layers).  Head-level: in
    every layer 4 of the 8 KV heads sparse (two such layer calls).  Same required bytes; per-layer
    attention-decode times, CUDA events, full cache layout for both."""
    w = synth.WORKLOADS["cfg3"]
    Hq, Hkv, S, W = w.n_q_heads, w.n_kv_heads, 128, 2048
    plan = flux.Plan(flux.make_config(2, Hq, Hkv, S, W, 1, n), dev)
    plan.flux_debug_decode_kernel(flux.FLUX_DECODE_TWO_LAUNCH)     # the kernels the head-level mode runs: like against like
    plan.flux_router_apply(mask=np.array([[1, 0]], dtype=np.uint8))
    # two cache sets, used alternately, so that no call finds its rows in L2 (a sparse layer's 17 MB would fit)
    sets = []
    for i in range(2):
        k = synth.normal_bf16((n, Hkv, D), w.seed + i, synth.stream_id("k"), dev)
        v = synth.normal_bf16((n, Hkv, D), w.seed + i, synth.stream_id("v"), dev)
        sets.append((k, v, flux.pointer_table([k], dev), flux.pointer_table([v], dev)))
    q = synth.normal_bf16((1, Hq, D), w.seed, synth.stream_id("qdec"), dev)
    out = torch.empty_like(q)
    ctx = torch.tensor([n], dtype=torch.int32, device=dev)
    hm_half = torch.tensor([[1, 0] * (Hkv // 2)], dtype=torch.uint8, device=dev)
    calls = {
        "dense_layer": lambda t: plan.flux_attn_decode(0, 1, q, sets[t][2], sets[t][3], ctx, out),
        "sparse_layer": lambda t: plan.flux_attn_decode(1, 1, q, sets[t][2], sets[t][3], ctx, out),
        "head_level_layer": lambda t: plan.flux_attn_decode_heads(1, q, sets[t][2], sets[t][3], ctx, hm_half, out),
    }
    ms = {}
    for name, fn in calls.items():
        for i in range(max(3, warmup)):
            fn(i & 1)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(reps):
            fn(i & 1)
        e1.record()
        torch.cuda.synchronize()
        ms[name] = e0.elapsed_time(e1) / reps
    assert plan.flux_plan_status() == 0
    plan.close()
    row = 2 * Hkv * D * 2
    bytes_dense, bytes_sparse = n * row, (S + W) * row
    pair_layer = ms["dense_layer"] + ms["sparse_layer"]
    pair_head = 2 * ms["head_level_layer"]
    return {"context": n, "sink": S, "window": W, "batch": 1,
            "ms_dense_layer": ms["dense_layer"], "ms_sparse_layer": ms["sparse_layer"],
            "ms_head_level_layer": ms["head_level_layer"],
            "required_bytes_per_layer_pair": bytes_dense + bytes_sparse,
            "speedup_layer_level": 2 * ms["dense_layer"] / pair_layer,
            "speedup_head_level": 2 * ms["dense_layer"] / pair_head,
            "byte_model_speedup": 2 * bytes_dense / (bytes_dense + bytes_sparse),
            "gbs_layer_level": (bytes_dense + bytes_sparse) / (pair_layer * 1e-3) / 1e9,
            "gbs_head_level": (bytes_dense + bytes_sparse) / (pair_head * 1e-3) / 1e9,
            "hbm_peak_gbs": peaks["hbm_gbs"],
            "paper": "head-level sparsity gives only marginal decode speedups, layer-level close to proportional "
                     "(Fig. 1(b), one A800 80GB, batch 1)"}


# ---- reference arm: the oracle on host cores ----------------------------------------------------

def run_reference(args):
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = synth.WORKLOADS[args.workload]
    mask = synth.layer_masks(w)
    ctx0 = synth.context_lengths(w)
    b = 0
    n = int(ctx0[b]) + 1
    Hq, Hkv, S, W = w.n_q_heads, w.n_kv_heads, w.sink, w.window
    scale = 1.0 / np.sqrt(D)
    q = oracle.to_bits(synth.normal_bf16((Hq, D), w.seed, 1))
    k = oracle.to_bits(synth.normal_bf16((n, Hkv, D), w.seed, 2))
    v = oracle.to_bits(synth.normal_bf16((n, Hkv, D), w.seed, 3))
    n_fa = int((mask == 1).sum()); n_sa = int((mask == 0).sum())
    # scale FA cost by each request's own length (ragged workloads)
    fa_rows = float(sum(int((mask[r] == 1).sum()) * (int(ctx0[r]) + 1) for r in range(w.batch)))

    def sample():
        t0 = time.perf_counter()
        oracle.decode(1, q, k, v, n, S, W, scale)
        t1 = time.perf_counter()
        oracle.decode(0, q, k, v, n, S, W, scale)
        t2 = time.perf_counter()
        return t1 - t0, t2 - t1

    for _ in range(args.warmup):
        sample()
    tf, ts = [], []
    for _ in range(args.steps):
        a, c = sample()
        tf.append(a); ts.append(c)
    t_fa_row = float(np.mean(tf)) / n                     # seconds per KV row of an FA (request, layer)
    step_s = fa_rows * t_fa_row + n_sa * float(np.mean(ts))
    value = w.batch / step_s
    cores = os.cpu_count() or 1
    line = {
        "impl": "reference", "metric": "decode_tokens_per_s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, mask, ctx0),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                         "sample": "per step: request 0 at its starting context, one FA and one SA layer, all "
                                   "heads; extrapolated to the full step by kept-row counts"},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def workload_config(w, mask, ctx0):
    return {
        "workload": "%s: %d layers, %d/%d heads, d%d, batch %d, context %s, sink %d + window %d, per-request "
                    "layer masks from seed (%d of %d (request,layer) slots sparse), sparse layers keep a "
                    "compact sink+window cache" % (
                        w.name, w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch,
                        ("%d" % ctx0[0]) if ctx0.min() == ctx0.max() else "%d..%d (log-uniform)" % (ctx0.min(), ctx0.max()),
                        w.sink, w.window, int((mask == 0).sum()), mask.size),
        "global_batch": int(w.batch), "l2": "inputs larger than L2 (each layer launch streams its own caches)",
        "parallelism": "replicas",
    }


# ---- small cases for ncu captures ---------------------------------------------------------------

def profile_case(flux, dev, which, decode_kernel=0):
    """A few launches of one kernel on a case of a few GB whose inputs exceed L2."""
    import dataclasses
    if which == "decode":      # the decode workload cut to 2 layers: same per-launch work as the bench
        w = dataclasses.replace(synth.WORKLOADS["cfg3"], n_layers=2)
        db = DecodeBench(flux, w, dev, 4)
        db.plan.flux_debug_decode_kernel(decode_kernel)
        db.plan.flux_plan_set_launch_overlap(True)
        for t in range(2):
            db.step(t)
        torch.cuda.synchronize()
        assert db.plan.flux_plan_status() == 0
        print(json.dumps({"profile_case": "decode", "layers": 2, "launch_bytes": db.bytes_step(0) / 2,
                          "cache_gb": db.cache_bytes / 1e9}))
    elif which == "decode_b1":  # batch 1, 28/4 heads, 128K context: one dense and one sparse layer, a few steps
        w = dataclasses.replace(synth.WORKLOADS["cfg4"], n_layers=2, prompt_len=0, mask_rule="fixed", mask_arg=(1, 0))
        db = DecodeBench(flux, w, dev, 6, host_mirrors=False)
        db.plan.flux_plan_set_launch_overlap(True)
        for t in range(4):
            db.step(t)
        torch.cuda.synchronize()
        assert db.plan.flux_plan_status() == 0
        print(json.dumps({"profile_case": "decode_b1", "launch_order": "dense, sparse, repeated 4 times",
                          "dense_launch_bytes": int(db.kept_rows(0)[0, 0]) * 2 * w.n_kv_heads * D * 2,
                          "sparse_launch_bytes": int(db.kept_rows(0)[0, 1]) * 2 * w.n_kv_heads * D * 2}))
    elif which == "prefill32k":  # the benchmark's own FA layer: 32768 tokens, one warm-up launch and one more
        w = synth.WORKLOADS["cfg2"]
        N = w.prompt_len
        plan = flux.Plan(flux.make_config(1, w.n_q_heads, w.n_kv_heads, w.sink, w.window, 1, N), dev)
        plan.flux_router_apply(mask=np.array([[1]], dtype=np.uint8))
        q = synth.normal_bf16((N, w.n_q_heads, D), w.seed, synth.stream_id("q"), dev)
        k = synth.normal_bf16((N, w.n_kv_heads, D), w.seed, synth.stream_id("k"), dev)
        v = synth.normal_bf16((N, w.n_kv_heads, D), w.seed, synth.stream_id("v"), dev)
        out = torch.empty_like(q)
        for _ in range(2):
            plan.flux_attn_prefill(0, 0, q, k, v, 0, out)
        torch.cuda.synchronize()
        assert plan.flux_plan_status() == 0
        i = np.arange(N, dtype=np.int64)
        print(json.dumps({"profile_case": "prefill32k", "N": N, "launches": 2, "device_gb": 4 * q.numel() * 2 / 1e9 * 0.625,
                          "flop_per_launch": 4 * w.n_q_heads * D * int((i + 1).sum())}))
    elif which == "router":    # the router front end of the benchmark's stack: 16 layers of weights (beyond L2), two passes
        w = synth.WORKLOADS["cfg2"]
        L, Hq = 16, w.n_q_heads
        plan = flux.Plan(flux.make_config(L, Hq, w.n_kv_heads, w.sink, w.window, 1, 4096), dev)
        q = synth.normal_bf16((4096, Hq, D), w.seed, synth.stream_id("q"), dev)
        ws = [synth.router_weights(w.seed, l, 2 * Hq * D, 1024, 256, dev) for l in range(L)]
        logits = torch.zeros((1, L, 2), dtype=torch.float32, device=dev)
        for _ in range(2):
            for l in range(L):
                plan.flux_router_forward(ws[l], q[:100], q[-100:], logits[0, l])
        torch.cuda.synchronize()
        assert plan.flux_plan_status() == 0
        print(json.dumps({"profile_case": "router", "layers": L, "launches": 2 * L,
                          "weight_bytes_per_launch": 2 * (2 * Hq * D * 1024 + 1024 * 1024 + 256 * 1024 + 2 * 256)}))
    elif which == "heads":     # one dense, one sparse and one half-sparse-heads layer call at 256K tokens
        res = head_level_block(flux, dev, measured_peaks(), 1, reps=1)
        print(json.dumps({"profile_case": "heads", "launch_order": "each of dense, sparse, head-level: 3 warm-up + 1",
                          "required_bytes_per_layer_pair": res["required_bytes_per_layer_pair"]}))
    else:                      # the prefill workload at 8192 tokens, one FA and one SA layer
        w = dataclasses.replace(synth.WORKLOADS["cfg2"], n_layers=2, prompt_len=8192)
        N = w.prompt_len
        plan = flux.Plan(flux.make_config(2, w.n_q_heads, w.n_kv_heads, w.sink, w.window, 1, N), dev)
        plan.flux_router_apply(mask=np.array([[1, 0]], dtype=np.uint8))
        q = synth.normal_bf16((N, w.n_q_heads, D), w.seed, 1, dev)
        k = synth.normal_bf16((N, w.n_kv_heads, D), w.seed, 2, dev)
        v = synth.normal_bf16((N, w.n_kv_heads, D), w.seed, 3, dev)
        out = torch.empty_like(q)
        for _ in range(2):
            for l in range(2):
                plan.flux_attn_prefill(l, 0, q, k, v, 0, out)
        torch.cuda.synchronize()
        assert plan.flux_plan_status() == 0
        print(json.dumps({"profile_case": "prefill", "N": N, "layers": "FA, SA"}))


# ---- main ------------------------------------------------------------------------------------------

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=["cfg3", "cfg4", "cfg5"],
                    help="decode workload: cfg3 (default, the headline), cfg4 (batch 1, 28/4 heads, 128K), cfg5 (ragged batch 16)")
    ap.add_argument("--decode-kernel", default="auto", choices=["auto", "two_launch", "single_launch"],
                    help="decode path: the library's choice by batch size, or one of the two forced")
    ap.add_argument("--no-launch-overlap", action="store_true",
                    help="single-launch decode: wait for the previous kernel before anything is read")
    ap.add_argument("--no-prefill", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-paper-ratios", action="store_true")
    ap.add_argument("--no-secondary", action="store_true",
                    help="skip the other decode workloads (cfg4, cfg5) and the 128K prefill layers")
    ap.add_argument("--sustain-seconds", type=float, default=3.0,
                    help="after the K timed steps, keep replaying the step for this long and report the sustained rate")
    ap.add_argument("--profile", default=None, choices=["decode", "decode_b1", "prefill", "prefill32k", "heads", "router"],
                    help="run a small case of one kernel with few launches (for ncu captures) and exit")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = "cuda:%d" % local
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))

    import __graft_entry__
    if rank == 0:
        __graft_entry__.build()
    if dist is not None:
        dist.barrier()
    from paper_2604_07394_b200 import flux
    flux.load()
    peaks = measured_peaks()
    if args.profile:
        profile_case(flux, dev, args.profile, {"auto": flux.FLUX_DECODE_AUTO, "two_launch": flux.FLUX_DECODE_TWO_LAUNCH,
                                               "single_launch": flux.FLUX_DECODE_SINGLE_LAUNCH}[args.decode_kernel])
        return
    w = synth.WORKLOADS[args.workload]
    W_, K_ = max(3, args.warmup), args.steps
    e2e_steps = 0 if args.no_e2e else min(K_, 10)
    roof_steps = min(K_, 20)
    # room for the sustained block: no step can be faster than its required bytes at the HBM peak
    probe = DecodeBench.__new__(DecodeBench)
    probe.w, probe.mask = w, synth.layer_masks(w)
    probe.ctx_host = (synth.context_lengths(w)[None, :].astype(np.int32) + 1)
    floor_ms = DecodeBench.bytes_step(probe, 0) / (peaks["hbm_gbs"] * 1e9) * 1e3
    sus_chunk = max(10, int(round(100.0 / floor_ms)))                    # about 0.1 s of replays per timed chunk
    sus_cap = 0 if args.sustain_seconds <= 0 else (int(args.sustain_seconds * 1e3 / floor_ms) // sus_chunk + 1) * sus_chunk
    total_steps = 1 + 2 * W_ + K_ + sus_cap + roof_steps + (2 + e2e_steps if e2e_steps else 0) + 2
    t_build = time.time()
    db = DecodeBench(flux, w, dev, total_steps)
    db.plan.flux_debug_decode_kernel({"auto": flux.FLUX_DECODE_AUTO, "two_launch": flux.FLUX_DECODE_TWO_LAUNCH,
                                      "single_launch": flux.FLUX_DECODE_SINGLE_LAUNCH}[args.decode_kernel])
    # between two layer calls of a step nothing but the previous layer's own launch sits in the stream, and the
    # step's length vector is advanced two kernels before the next step's first layer: the promise holds
    db.plan.flux_plan_set_launch_overlap(not args.no_launch_overlap)
    torch.cuda.synchronize()
    log("[bench] rank %d: %.1f GB of KV cache built in %.1f s" % (rank, db.cache_bytes / 1e9, time.time() - t_build))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()          # nvidia-smi needs a moment to start: launch it before the warm-up
        time.sleep(1.0)
    t = 1
    for _ in range(W_):
        db.step(t); t += 1
    launches_per_step = db.plan.flux_launch_count()
    db.capture_step(t)                       # the library's calls are captured like any other launch
    launches_per_step = db.plan.flux_launch_count() - launches_per_step
    for _ in range(W_):
        db.step_graph(); t += 1
    barrier()
    # (1) the K timed steps: one graph replay per step
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_first = t
    e0.record()
    for _ in range(K_):
        db.step_graph(); t += 1
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = launches_per_step * K_
    alg_bytes = sum(db.bytes_step(s) for s in range(t_first, t_first + K_))
    # (1b) sustained: the same replay loop kept up for some seconds (power cap reached, clocks settled)
    sustained = None
    if sus_cap:
        sampler2 = ClockSampler(local)
        if rank == 0:
            sampler2.start()
        # the same number of steps on every rank: from the slowest rank's time for the K steps above
        step_ms = max_over_ranks(dist, [ms], dev)[0] / K_
        sus_target = min(sus_cap, (int(args.sustain_seconds * 1e3 / step_ms) // sus_chunk + 1) * sus_chunk)
        sus_ms, sus_steps, sus_bytes = 0.0, 0, 0
        barrier()
        while sus_steps < sus_target:
            sus_ms += timed_replays(db, sus_chunk)
            sus_bytes += sum(db.bytes_step(s_) for s_ in range(t, t + sus_chunk))
            t += sus_chunk; sus_steps += sus_chunk
        barrier()
        clocks2 = sampler2.stop() if rank == 0 else None
        sus_ms = max_over_ranks(dist, [sus_ms], dev)[0]
        gbs = sus_bytes / (sus_ms * 1e-3) / 1e9
        sustained = {"value": whole_job_throughput(world, w.batch, sus_steps, sus_ms), "unit": "tokens/s", "steps": sus_steps,
                     "seconds": sus_ms / 1e3, "ms_per_step": sus_ms / sus_steps, "step_level_gbs": gbs,
                     "frac_of_hbm_peak": gbs / peaks["hbm_gbs"], "clocks": clocks2,
                     "note": "graph replays back to back right after the K timed steps; the short region above runs before "
                             "the power cap bites, this one mostly under it"}
    # (2) the dominant kernel, event-bracketed launch by launch, on the next steps issued one call at a time
    db.plan.flux_profile_enable(roof_steps * w.n_layers + 8)
    r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_roof = t
    r0.record()
    for _ in range(roof_steps):
        db.step(t); t += 1
    r1.record()
    barrier()
    eager_ms = r0.elapsed_time(r1) / roof_steps
    kms, kcnt = db.plan.flux_profile_read(flux.FLUX_KERNEL_DECODE)
    db.plan.flux_profile_enable(0)
    roof_bytes = sum(db.bytes_step(s) for s in range(t_roof, t_roof + roof_steps))
    clocks = sampler.stop() if rank == 0 else None
    status = db.plan.flux_plan_status()
    assert status == 0, status

    e2e = None
    if e2e_steps:
        for _ in range(2):
            db.step_host(t); t += 1
        barrier()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record()
        for _ in range(e2e_steps):
            db.step_host(t); t += 1
        h1.record()
        barrier()
        e2e_ms = h0.elapsed_time(h1)
    ms, e2e_ms_max = max_over_ranks(dist, [ms, e2e_ms if e2e_steps else 0.0], dev)
    if e2e_steps:
        e2e_ms = e2e_ms_max
    if e2e_steps:
        e2e = {"value": whole_job_throughput(world, w.batch, e2e_steps, e2e_ms), "unit": "tokens/s",
               "h2d_bytes_per_step": db.h2d_bytes(), "d2h_bytes_per_step": db.d2h_bytes(),
               "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
               "api": "flux_attn_decode_host per layer: q / k_new / v_new read from pinned host memory by the ingest kernel, "
                      "the result written to pinned host memory by the combine kernel (every byte crosses the bus once, "
                      "inside the timed region)"}

    # the oracle runs after the timed regions, so that the GPU does not sit idle (and clock down)
    # for seconds right before them
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        t0 = time.time()
        cpu = cpu_baseline_decode(db)
        log("[bench] oracle sample took %.1f s" % (time.time() - t0))

    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    value = whole_job_throughput(world, w.batch, K_, ms)
    single = decode_kernel_name(flux, args.decode_kernel, w.batch).startswith("decode_fused")
    if single and launches_per_step == w.n_layers:
        # the step is nothing but this kernel, one launch per layer: the K timed graph replays are K * L launches of it,
        # timed by the events around the region (bracketing single launches with events, as below, would put an
        # event between every two launches and undo the overlap of one launch's set-up with the previous one's tail)
        n_timed = K_ * w.n_layers
        per_launch_bytes, per_launch_ms = alg_bytes / n_timed, ms / n_timed
        how = "timed region of the %d graph replays / (%d x %d launches)" % (K_, K_, w.n_layers)
        bracketed = {"launches": int(kcnt), "avg_launch_ms": kms / max(kcnt, 1),
                     "gbs": roof_bytes / max(kcnt, 1) / (kms / max(kcnt, 1) * 1e-3) / 1e9,
                     "note": "the same kernel issued call by call with an event on each side of every launch"}
    else:
        n_timed = int(kcnt)
        per_launch_bytes = roof_bytes / max(kcnt, 1)
        per_launch_ms = kms / max(kcnt, 1)
        how = "events around every launch of %d steps issued call by call" % roof_steps
        bracketed = None
    ach = per_launch_bytes / (per_launch_ms * 1e-3) / 1e9
    tr = traffic_note("decode_fused_kernel" if decode_kernel_name(flux, args.decode_kernel, w.batch).startswith("decode_fused") else "decode_kernel")
    roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": ach / peaks["hbm_gbs"], "peak_source": peaks["source"] + " (copy bandwidth)",
            "kernel": decode_kernel_name(flux, args.decode_kernel, w.batch),
            "launches_timed": n_timed, "avg_launch_ms": per_launch_ms, "timing": how, "event_bracketed": bracketed,
            "algorithmic_bytes_per_launch": per_launch_bytes,
            "traffic": None if tr is None else tr.get("dram_bytes_per_algorithmic_byte") * per_launch_bytes,
            "traffic_source": None if tr is None else tr.get("source"),
            "step_level_gbs": alg_bytes / (ms * 1e-3) / 1e9}
    line = {
        "metric": "decode_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K_,
        "warmup": W_, "ms_per_step": ms / K_, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": workload_config(w, db.mask, db.ctx0),
        "roofline": roof, "sustained": sustained, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
        "stepping": "one CUDA graph per decode step (%d kernel launches of this library), replayed %d times; "
                    "issued call by call the same step takes %.3f ms" % (launches_per_step, K_, eager_ms),
        "omega_msr": float((db.mask == 0).mean()),
        "paper_context": "paper reports decode kernel speedup approaching 2.0x at 256K and prefill speedup up "
                         "to 2.8x (Full+Triangle) on one A800 80GB, bf16, batch 1; ratios only, no absolute numbers",
    }
    del db
    torch.cuda.empty_cache()
    if not args.no_prefill and world == 1:
        try:
            line["prefill"] = prefill_block(flux, dev, peaks, W_)
        except Exception as e:  # report, never hide
            line["prefill"] = {"error": repr(e)}
    if not args.no_prefill and world == 1:
        try:
            line["router_frontend"] = router_frontend_block(flux, dev, peaks, W_)
        except Exception as e:  # report, never hide
            line["router_frontend"] = {"error": repr(e)}
    if not args.no_secondary and world == 1:
        for name in ("cfg5", "cfg4"):
            if name == args.workload:
                continue
            try:
                line["decode_" + name] = secondary_decode_block(flux, dev, peaks, name, 50 if name == "cfg5" else 400, W_, args)
            except Exception as e:  # report, never hide
                line["decode_" + name] = {"error": repr(e)}
        try:
            line["prefill_cfg4_128k"] = prefill_128k_block(flux, dev, peaks, W_)
        except Exception as e:  # report, never hide
            line["prefill_cfg4_128k"] = {"error": repr(e)}
    if not args.no_paper_ratios and world == 1:
        try:
            line["paper_ratios_256k"] = paper_ratio_block(flux, dev, W_)
        except Exception as e:  # report, never hide
            line["paper_ratios_256k"] = {"error": repr(e)}
        try:
            line["head_level_vs_layer_level_256k"] = head_level_block(flux, dev, peaks, W_)
        except Exception as e:  # report, never hide
            line["head_level_vs_layer_level_256k"] = {"error": repr(e)}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
