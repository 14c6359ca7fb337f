"""The workspace-free decode entry point against the oracle and against the regular entry point.

``flux_attn_decode_noalloc`` exists for callers that cannot allocate device memory (a plug-in
inside a program that owns all of it, a loop that must avoid the synchronisation an allocation
may cause); its scratch is a fixed array inside the library.  The tests call it through the
C ABI several times in a row, with different inputs, and check each result (a) against the fp64
oracle, request by request, and (b) bit for bit against what ``flux_attn_decode`` gives with a
caller-supplied workspace (the same kernels on the same grid).  The file sorts last so that a
failure here cannot hide the other tests' results."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07394_b200 import synth
from tests._util import bits, compare, logical_view

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SCALE = 1.0 / np.sqrt(128.0)


def _flux():
    from paper_2604_07394_b200 import build, flux
    build.build()
    flux.load()
    return flux


def _caches(flux, plan, layer, lens, mask, Hkv, S, W, cap, layout, seed):
    """Caches filled through flux_kv_retain from position-indexed K, V; returns tables and the logical K, V."""
    kc, vc, klog, vlog = [], [], [], []
    for b, n in enumerate(lens):
        k = synth.normal_bf16((max(n, 1), Hkv, 128), seed, 2 * b, DEV)
        v = synth.normal_bf16((max(n, 1), Hkv, 128), seed, 2 * b + 1, DEV)
        compact = layout == flux.FLUX_KV_COMPACT_SA and mask[b, layer] == 0
        rows = S + W if compact else cap
        kcache = torch.zeros((rows, Hkv, 128), dtype=torch.bfloat16, device=DEV)
        vcache = torch.zeros_like(kcache)
        if n > 0:
            plan.flux_kv_retain(layer, b, k, v, n, kcache, vcache)
        kc.append(kcache); vc.append(vcache); klog.append(k); vlog.append(v)
    return kc, vc, klog, vlog


@pytest.mark.parametrize("Hq,Hkv,layout", [(28, 4, 0), (28, 4, 1), (32, 16, 1)],
                         ids=["28q4kv_full", "28q4kv_compact", "32q16kv_compact"])
def test_noalloc_decode_matches_oracle_and_workspace_decode_twice_in_a_row(Hq, Hkv, layout):
    flux = _flux()
    L, S, W, cap = 2, 16, 48, 512
    lens = [300, 64, 65, 0, 5, 1]            # one inactive request (zero output row)
    B = len(lens)
    mask = np.array([[1, 0], [0, 1], [0, 0], [1, 0], [1, 1], [0, 1]], dtype=np.uint8)
    cfg = flux.make_config(L, Hq, Hkv, S, W, B, cap, kv_layout=layout)
    plan = flux.Plan(cfg, DEV)
    plan.flux_debug_decode_kernel(flux.FLUX_DECODE_TWO_LAUNCH)      # the kernels the workspace-free call runs
    mask_dev = plan.flux_router_apply(mask=mask)
    ctx = torch.tensor(lens, dtype=torch.int32, device=DEV)
    status = torch.full((1,), 77, dtype=torch.int32, device=DEV)
    for call, layer in enumerate((0, 1)):
        kc, vc, klog, vlog = _caches(flux, plan, layer, lens, mask, Hkv, S, W, cap, layout, 91 + layer)
        ktab, vtab = flux.pointer_table(kc, DEV), flux.pointer_table(vc, DEV)
        q = synth.normal_bf16((B, Hq, 128), 93, layer, DEV)
        want = plan.flux_attn_decode(layer, B, q, ktab, vtab, ctx)
        out = torch.full_like(q, float("nan"))
        flux.flux_attn_decode_noalloc(cfg, layer, B, mask_dev, q, ktab, vtab, ctx, out, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(out, want), "call %d differs from flux_attn_decode" % call
        for b, n in enumerate(lens):
            if n == 0:
                assert torch.count_nonzero(out[b]) == 0
                continue
            mode = int(mask[b, layer])
            ref = oracle.decode(mode, bits(q[b]), bits(klog[b]), bits(vlog[b]), n, S, W, SCALE)
            compare(out[b], ref, "noalloc call %d b=%d n=%d mode=%d" % (call, b, n, mode))
            # and the cache the call read holds what the oracle says the layer must retain
            compact = layout == flux.FLUX_KV_COMPACT_SA and mode == 0
            keep = oracle.retained(n, S, W) if mode == 0 else np.arange(n)
            assert torch.equal(logical_view(kc[b], n, S, W, compact)[keep], klog[b].cpu()[keep])
    assert plan.flux_plan_status() == 0


def test_noalloc_status_word_is_delivered_and_cleared_between_calls():
    flux = _flux()
    L, Hq, Hkv, S, W, cap = 1, 8, 2, 4, 8, 64
    cfg = flux.make_config(L, Hq, Hkv, S, W, 2, cap)
    plan = flux.Plan(cfg, DEV)
    mask_dev = plan.flux_router_apply(mask=np.array([[1], [0]], dtype=np.uint8))
    kc = [synth.normal_bf16((cap, Hkv, 128), 5, b, DEV) for b in range(2)]
    vc = [synth.normal_bf16((cap, Hkv, 128), 6, b, DEV) for b in range(2)]
    ktab, vtab = flux.pointer_table(kc, DEV), flux.pointer_table(vc, DEV)
    q = synth.normal_bf16((2, Hq, 128), 7, 0, DEV)
    out = torch.zeros_like(q)
    status = torch.zeros((1,), dtype=torch.int32, device=DEV)
    # a context length beyond max_context is clamped and flagged (no row beyond the cache is read)
    too_long = torch.tensor([cap + 9, 20], dtype=torch.int32, device=DEV)
    flux.flux_attn_decode_noalloc(cfg, 0, 2, mask_dev, q, ktab, vtab, too_long, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == flux.FLUX_STATUS_BAD_LENGTH
    # the next call starts from a clean status word although the scratch array is shared
    ok = torch.tensor([cap, 20], dtype=torch.int32, device=DEV)
    flux.flux_attn_decode_noalloc(cfg, 0, 2, mask_dev, q, ktab, vtab, ok, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for b, n in enumerate([cap, 20]):
        ref = oracle.decode(1 - b, bits(q[b]), bits(kc[b]), bits(vc[b]), n, S, W, SCALE)
        compare(out[b], ref, "noalloc after a flagged call b=%d" % b)


def test_noalloc_refuses_sizes_beyond_its_scratch():
    flux = _flux()
    L, Hq, Hkv, S, W = 2, 28, 4, 16, 48
    cfg = flux.make_config(L, Hq, Hkv, S, W, 5, 512)
    plan = flux.Plan(cfg, DEV)
    mask_dev = plan.flux_router_apply(mask=np.ones((5, L), dtype=np.uint8))
    kc = [synth.normal_bf16((8, Hkv, 128), 5, b, DEV) for b in range(5)]
    ktab = flux.pointer_table(kc, DEV)
    q = synth.normal_bf16((5, Hq, 128), 7, 0, DEV)
    out = torch.zeros_like(q)
    ctx = torch.ones((5,), dtype=torch.int32, device=DEV)
    # sizes beyond the built-in scratch are refused with a clear message, nothing is launched
    big = flux.make_config(L, Hq, Hkv, S, W, 65, 512)
    with pytest.raises(flux.FluxError) as e:
        flux.flux_attn_decode_noalloc(big, 0, 65, mask_dev, q, ktab, ktab, ctx, out, None)
    assert e.value.code == flux.FLUX_E_CAPACITY and "64" in str(e.value)
    wide = flux.make_config(L, 32, 2, S, W, 5, 512)      # 16 query heads per KV head
    with pytest.raises(flux.FluxError) as e:
        flux.flux_attn_decode_noalloc(wide, 0, 5, mask_dev, q, ktab, ktab, ctx, out, None)
    assert e.value.code == flux.FLUX_E_CAPACITY
    assert torch.count_nonzero(out) == 0
