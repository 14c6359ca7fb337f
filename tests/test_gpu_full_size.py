"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times, on sampled
outputs the oracle computes one by one (boundary rows of the kept sets, tile edges, random rows;
first / last heads of GQA groups).  Dispatch records are compared bit-exactly."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2604_07394_b200 import synth
from tests._util import bits, compact_rows_to_positions, compare, expand_ranges

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SCALE = 1.0 / np.sqrt(128.0)


@pytest.fixture(scope="module")
def flux():
    from paper_2604_07394_b200 import build, flux as f
    build.build()
    f.load()
    return f


def _sample_heads(Hq, G):
    return sorted({0, G - 1, G, Hq // 2, Hq - G, Hq - 1} & set(range(Hq)))


@pytest.mark.parametrize("cfg", ["cfg2", "cfg4"])
def test_prefill_full_size_sampled_rows(flux, cfg):
    """cfg2: 32K tokens, 32/8 heads, sink 128 + window 2048; cfg4: 128K tokens, 28/4 heads (7 query
    heads per KV head), sink 128 + window 4096.  One FA and one SA layer each, whole prompt in one
    call (as the benchmark does) and, for cfg2, also in chunks of 16384 (Appendix D.3 chunk size)."""
    w = synth.WORKLOADS[cfg]
    N, Hq, Hkv, S, W = w.prompt_len, w.n_q_heads, w.n_kv_heads, w.sink, w.window
    plan = flux.Plan(flux.make_config(2, Hq, Hkv, S, W, 1, N), DEV)
    plan.flux_router_apply(mask=np.array([[1, 0]], dtype=np.uint8))
    q = synth.normal_bf16((N, Hq, 128), w.seed, synth.stream_id("q"), DEV)
    k = synth.normal_bf16((N, Hkv, 128), w.seed, synth.stream_id("k"), DEV)
    v = synth.normal_bf16((N, Hkv, 128), w.seed, synth.stream_id("v"), DEV)
    rows = synth.sample_rows(N, S, W, 40, w.seed)
    heads = _sample_heads(Hq, Hq // Hkv)
    rr = np.repeat(rows, len(heads))
    hh = np.tile(np.asarray(heads, dtype=np.int64), len(rows))
    qb, kb, vb = bits(q), bits(k), bits(v)
    for layer, mode in ((0, oracle.FA), (1, oracle.SA)):
        ref = oracle.prefill_rows(mode, qb, kb, vb, 0, rr, hh, S, W, SCALE)
        out = plan.flux_attn_prefill(layer, 0, q, k, v, 0)
        rec = plan.flux_debug_dispatch(1)
        got = out[torch.from_numpy(rr).to(DEV), torch.from_numpy(hh).to(DEV)]
        compare(got, ref, "%s prefill mode %d" % (cfg, mode))
        assert rec[0, 0] == mode and rec[0, 3] == N
        assert expand_ranges(rec[0]) == oracle.kept(mode, N - 1, S, W).tolist()
        if cfg == "cfg2":
            out2 = torch.empty_like(q)
            for a in range(0, N, 16384):
                out2[a:a + 16384] = plan.flux_attn_prefill(layer, 0, q[a:a + 16384], k[:a + 16384], v[:a + 16384], a)
            got2 = out2[torch.from_numpy(rr).to(DEV), torch.from_numpy(hh).to(DEV)]
            compare(got2, ref, "%s chunked prefill mode %d" % (cfg, mode))
    assert plan.flux_plan_status() == 0


def test_prefill_256k_in_chunks_sampled_rows(flux):
    """The paper's headline length (Sec. 4.3: 256K tokens): Llama-3-8B attention shapes, sink 128 +
    window 2048 (Table 3), prefilled in chunks of 16384 queries (Appendix D.3), one FA and one SA
    layer; sampled rows of every chunk region against the oracle."""
    N, Hq, Hkv, S, W, C = 262144, 32, 8, 128, 2048, 16384
    plan = flux.Plan(flux.make_config(2, Hq, Hkv, S, W, 1, N), DEV)
    plan.flux_router_apply(mask=np.array([[1, 0]], dtype=np.uint8))
    q = synth.normal_bf16((N, Hq, 128), 606, synth.stream_id("q"), DEV)
    k = synth.normal_bf16((N, Hkv, 128), 606, synth.stream_id("k"), DEV)
    v = synth.normal_bf16((N, Hkv, 128), 606, synth.stream_id("v"), DEV)
    rows = np.unique(np.concatenate([synth.sample_rows(N, S, W, 12, 606),
                                     np.array([C - 1, C, 5 * C + 77, N - C, N - C - 1])]))
    heads = [0, 3, 4, 31]
    rr = np.repeat(rows, len(heads))
    hh = np.tile(np.asarray(heads, dtype=np.int64), len(rows))
    qb, kb, vb = bits(q), bits(k), bits(v)
    out = torch.empty_like(q)
    for layer, mode in ((1, oracle.SA), (0, oracle.FA)):
        for a in range(0, N, C):
            plan.flux_attn_prefill(layer, 0, q[a:a + C], k[:a + C], v[:a + C], a, out[a:a + C])
        ref = oracle.prefill_rows(mode, qb, kb, vb, 0, rr, hh, S, W, SCALE)
        compare(out[torch.from_numpy(rr).to(DEV), torch.from_numpy(hh).to(DEV)], ref, "256K prefill mode %d" % mode)
    assert plan.flux_plan_status() == 0


@pytest.mark.parametrize("cfg,dk", [("cfg3", 0), ("cfg3", 1), ("cfg3", 3), ("cfg4", 0), ("cfg4", 1), ("cfg4", 3), ("cfg5", 1), ("cfg5", 3)],
                         ids=["cfg3", "cfg3_two_launch", "cfg3_overlap", "cfg4", "cfg4_two_launch", "cfg4_overlap", "cfg5_two_launch",
                              "cfg5_overlap"])
def test_decode_full_size_sampled(flux, cfg, dk):
    """The decode workloads as bench.py builds them (compact sparse caches, per-request masks,
    ragged lengths for cfg5): two steps; at each, for every request two FA and two SA layers are
    checked against the oracle on sampled heads, and every request's dispatch record on those
    layers is compared with the oracle's kept set."""
    import bench

    w = synth.WORKLOADS[cfg]
    if cfg == "cfg4":       # decode phase of the 128K workload: the cache is drawn directly
        w = dataclasses.replace(w, prompt_len=0)
    db = bench.DecodeBench(flux, w, DEV, 4)
    db.plan.flux_debug_decode_kernel(min(dk, 2))     # 0: the default choice for the batch size; 1 / 2: the other kernel
    db.plan.flux_plan_set_launch_overlap(dk == 3)    # 3: single launch with launch overlap
    heads = _sample_heads(w.n_q_heads, w.n_q_heads // w.n_kv_heads)
    S, W = w.sink, w.window
    for t in (0, 1):
        db.step(t)
        torch.cuda.synchronize()
        for b in range(w.batch):
            n = int(db.ctx_host[t][b])
            for mode in (1, 0):
                for l in np.nonzero(db.mask[b] == mode)[0][[0, -1]]:
                    l = int(l)
                    compact = mode == 0
                    kl = bench.logical_cache(db.kc[l][b].cpu(), n, S, W, compact)
                    vl = bench.logical_cache(db.vc[l][b].cpu(), n, S, W, compact)
                    ref = oracle.decode(mode, bits(db.q[l, b]), bits(kl), bits(vl), n, S, W, SCALE,
                                        heads=np.asarray(heads, dtype=np.int64))
                    compare(db.out[l, b][heads], ref, "%s decode t=%d b=%d l=%d mode=%d" % (cfg, t, b, l, mode))
        # dispatch of the last layer launched, every request
        l = w.n_layers - 1
        rec = db.plan.flux_debug_dispatch(w.batch)
        for b in range(w.batch):
            n = int(db.ctx_host[t][b])
            mode = int(db.mask[b, l])
            assert rec[b, 0] == mode and rec[b, 2] == b and rec[b, 3] == n
            rows = expand_ranges(rec[b])
            want = oracle.kept(mode, n - 1, S, W).tolist()
            assert (compact_rows_to_positions(rows, n, S, W) if mode == 0 else rows) == want
    assert db.plan.flux_plan_status() == 0


def test_sparse_outputs_ignore_keys_outside_the_kept_set_at_full_size(flux):
    """A property that needs no oracle and holds at any size: changing K and V at positions a query does
    not keep must leave its output bit-identical.  32K prefill and a 64K
    decode in the full cache layout; the FA layer, which keeps those positions, must change."""
    w = synth.WORKLOADS["cfg2"]
    N, Hq, Hkv, S, W = w.prompt_len, w.n_q_heads, w.n_kv_heads, w.sink, w.window
    plan = flux.Plan(flux.make_config(2, Hq, Hkv, S, W, 1, 65536 + 8), DEV)
    plan.flux_router_apply(mask=np.array([[1, 0]], dtype=np.uint8))
    q = synth.normal_bf16((N, Hq, 128), w.seed, synth.stream_id("q"), DEV)
    k = synth.normal_bf16((N, Hkv, 128), w.seed, synth.stream_id("k"), DEV)
    v = synth.normal_bf16((N, Hkv, 128), w.seed, synth.stream_id("v"), DEV)
    a, b = 5000, 6000                                   # positions [a, b) are rewritten
    k2, v2 = k.clone(), v.clone()
    k2[a:b] = synth.normal_bf16((b - a, Hkv, 128), 99, 1, DEV)
    v2[a:b] = synth.normal_bf16((b - a, Hkv, 128), 99, 2, DEV)
    first_unaffected = b - 1 + W                        # the first query whose window starts after b - 1
    sa0, sa1 = plan.flux_attn_prefill(1, 0, q, k, v, 0), plan.flux_attn_prefill(1, 0, q, k2, v2, 0)
    assert torch.equal(sa0[:a].view(torch.int16), sa1[:a].view(torch.int16))
    assert torch.equal(sa0[first_unaffected:].view(torch.int16), sa1[first_unaffected:].view(torch.int16))
    assert not torch.equal(sa0[a:first_unaffected].view(torch.int16), sa1[a:first_unaffected].view(torch.int16))
    fa0, fa1 = plan.flux_attn_prefill(0, 0, q, k, v, 0), plan.flux_attn_prefill(0, 0, q, k2, v2, 0)
    assert torch.equal(fa0[:a].view(torch.int16), fa1[:a].view(torch.int16))
    changed = (fa0[b:] != fa1[b:]).flatten(1).any(dim=1)
    assert bool(changed.all())                      # every later FA row sees the rewritten keys
    # decode at 65536 tokens, full layout: rewrite everything between the sink and the window
    n = 65536
    kc = synth.normal_bf16((n, Hkv, 128), 7, 1, DEV)
    vc = synth.normal_bf16((n, Hkv, 128), 7, 2, DEV)
    kc2, vc2 = kc.clone(), vc.clone()
    kc2[S:n - W] = synth.normal_bf16((n - W - S, Hkv, 128), 98, 1, DEV)
    vc2[S:n - W] = synth.normal_bf16((n - W - S, Hkv, 128), 98, 2, DEV)
    qd = synth.normal_bf16((1, Hq, 128), 7, 3, DEV)
    ctx = torch.tensor([n], dtype=torch.int32, device=DEV)
    outs = []
    for kk, vv in ((kc, vc), (kc2, vc2)):
        kt, vt = flux.pointer_table([kk], DEV), flux.pointer_table([vv], DEV)
        outs.append((plan.flux_attn_decode(1, 1, qd, kt, vt, ctx).clone(), plan.flux_attn_decode(0, 1, qd, kt, vt, ctx).clone()))
    assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16))          # SA: identical
    assert not torch.equal(outs[0][1].view(torch.int16), outs[1][1].view(torch.int16))      # FA: differs
    assert plan.flux_plan_status() == 0
