"""A decode step evaluated in pieces over disjoint key ranges (flux_attn_decode_partial) and merged
(flux_attn_combine): against the fp64 oracle, against the oracle's own merge rule applied to the
pieces, and against the single-call result."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07394_b200 import keysplit, synth
from tests._util import bits, compare

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SCALE = 1.0 / np.sqrt(128.0)
LN2 = float(np.log(2.0))


@pytest.fixture(scope="module")
def flux():
    from paper_2604_07394_b200 import build, flux as f
    build.build()
    f.load()
    return f


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("layout", [0, 1])
def test_pieces_over_key_ranges_merge_to_the_whole_step(flux, layout, world):
    Hq, Hkv, S, W, L = 8, 2, 16, 48, 2
    lens = [3000, 500, 37, 1, 0, 64]                     # incl. a request shorter than a range and an inactive one
    B = len(lens)
    cap = 3008
    mask = np.array([[1, 0], [0, 1], [1, 1], [0, 0], [1, 0], [0, 1]], dtype=np.uint8)
    plan = flux.Plan(flux.make_config(L, Hq, Hkv, S, W, B, cap, kv_layout=layout), DEV)
    plan.flux_router_apply(mask=mask)
    ranges = keysplit.key_ranges(lens, world)
    assert (ranges[0, :, 0] == 0).all() and (ranges[-1, :, 1] == np.asarray(lens)).all()
    assert (ranges[1:, :, 0] == ranges[:-1, :, 1]).all()
    ctx = torch.tensor(lens, dtype=torch.int32, device=DEV)
    for layer in range(L):
        kc, vc, klog, vlog = [], [], [], []
        for b, n in enumerate(lens):
            k = synth.normal_bf16((max(n, 1), Hkv, 128), 31, 10 * layer + b, DEV)
            v = synth.normal_bf16((max(n, 1), Hkv, 128), 32, 10 * layer + b, DEV)
            compact = layout == 1 and mask[b, layer] == 0
            kcache = torch.zeros((S + W if compact else cap, Hkv, 128), dtype=torch.bfloat16, device=DEV)
            vcache = torch.zeros_like(kcache)
            if n > 0:
                plan.flux_kv_retain(layer, b, k, v, n, kcache, vcache)
            kc.append(kcache); vc.append(vcache); klog.append(k); vlog.append(v)
        kt, vt = flux.pointer_table(kc, DEV), flux.pointer_table(vc, DEV)
        q = synth.normal_bf16((B, Hq, 128), 33, layer, DEV)
        pieces_o, pieces_ml = [], []
        for r in range(world):
            kb = torch.from_numpy(ranges[r, :, 0].copy()).to(DEV)
            ke = torch.from_numpy(ranges[r, :, 1].copy()).to(DEV)
            po, pml = plan.flux_attn_decode_partial(layer, B, q, kt, vt, ctx, kb, ke)
            pieces_o.append(po); pieces_ml.append(pml)
        po_all, pml_all = torch.stack(pieces_o), torch.stack(pieces_ml)
        out = plan.flux_attn_combine(B, po_all, pml_all)
        whole = plan.flux_attn_decode(layer, B, q, kt, vt, ctx)
        po_h, pml_h = po_all.cpu().numpy().astype(np.float64), pml_all.cpu().numpy().astype(np.float64)
        for b, n in enumerate(lens):
            if n == 0:
                assert torch.count_nonzero(out[b]) == 0 and (pml_h[:, b, :, 1] == 0).all()
                continue
            mode = int(mask[b, layer])
            ref = oracle.decode(mode, bits(q[b]), bits(klog[b]), bits(vlog[b]), n, S, W, SCALE)
            compare(out[b], ref, "merged pieces b=%d n=%d mode=%d" % (b, n, mode))
            compare(whole[b], ref, "single call b=%d" % b)
            # the oracle's merge rule on the pieces (normalised outputs, natural-log maxima) gives the same row
            for h in range(Hq):
                m, l, o = -np.inf, 0.0, np.zeros(128)
                for r in range(world):
                    lp = pml_h[r, b, h, 1]
                    if lp == 0.0:
                        continue
                    mp, op = pml_h[r, b, h, 0] * LN2, po_h[r, b, h] / lp
                    m, l, o = (mp, lp, op) if l == 0.0 else oracle.merge(m, l, o, mp, lp, op)
                compare(out[b, h], o[None, :], "oracle merge of the pieces b=%d h=%d" % (b, h))
            # a sparse request (beyond sink + window) is taken whole by the range that holds its newest position
            if mode == 0 and n > S + W:
                owners = [r for r in range(world) if pml_h[r, b, 0, 1] > 0]
                assert owners == [r for r in range(world) if ranges[r, b, 0] <= n - 1 < ranges[r, b, 1]]
    assert plan.flux_plan_status() == 0


def test_partial_call_argument_errors(flux):
    plan = flux.Plan(flux.make_config(1, 8, 2, 4, 8, 2, 64), DEV)
    plan.flux_router_apply(mask=np.array([[1], [0]], dtype=np.uint8))
    kc = [synth.normal_bf16((64, 2, 128), 1, b, DEV) for b in range(2)]
    kt = flux.pointer_table(kc, DEV)
    q = synth.normal_bf16((2, 8, 128), 2, 0, DEV)
    ctx = torch.tensor([10, 10], dtype=torch.int32, device=DEV)
    host_range = torch.zeros(2, dtype=torch.int32)      # key ranges must live on the device
    with pytest.raises(flux.FluxError) as e:
        plan.flux_attn_decode_partial(0, 2, q, kt, kt, ctx, host_range, host_range)
    assert e.value.code == flux.FLUX_E_INVALID_ARG
    po = torch.zeros((2, 2, 8, 128), dtype=torch.float32, device=DEV)
    pml = torch.zeros((2, 2, 8, 2), dtype=torch.float32, device=DEV)
    with pytest.raises(flux.FluxError) as e:
        plan.flux_attn_combine(3, po, pml)              # beyond the plan's max_batch
    assert e.value.code == flux.FLUX_E_CAPACITY


def _split_case(flux, layout, lens, mask, world, L=2):
    Hq, Hkv, S, W = 8, 2, 16, 48
    B, cap = len(lens), 3008
    plan = flux.Plan(flux.make_config(L, Hq, Hkv, S, W, B, cap, kv_layout=layout), DEV)
    plan.flux_router_apply(mask=mask)
    ranges = keysplit.key_ranges(lens, world)
    ctx = torch.tensor(lens, dtype=torch.int32, device=DEV)
    layers = []
    for layer in range(L):
        kc, vc, klog, vlog = [], [], [], []
        for b, n in enumerate(lens):
            k = synth.normal_bf16((max(n, 1), Hkv, 128), 41, 10 * layer + b, DEV)
            v = synth.normal_bf16((max(n, 1), Hkv, 128), 42, 10 * layer + b, DEV)
            compact = layout == 1 and mask[b, layer] == 0
            kcache = torch.zeros((S + W if compact else cap, Hkv, 128), dtype=torch.bfloat16, device=DEV)
            vcache = torch.zeros_like(kcache)
            if n > 0:
                plan.flux_kv_retain(layer, b, k, v, n, kcache, vcache)
            kc.append(kcache); vc.append(vcache); klog.append(k); vlog.append(v)
        layers.append((flux.pointer_table(kc, DEV), flux.pointer_table(vc, DEV), kc, vc, klog, vlog,
                       synth.normal_bf16((B, Hq, 128), 43, layer, DEV)))
    return plan, ranges, ctx, layers, (Hq, Hkv, S, W, B)


@pytest.mark.parametrize("world", [2, 4])
@pytest.mark.parametrize("layout", [0, 1])
def test_pushed_pieces_and_waiting_merge_with_the_ranks_emulated_on_one_gpu(flux, layout, world):
    """The exchange without a library call: every rank's merge kernel stores its piece into every rank's gather
    buffer and raises that rank's flag; every rank's merge waits for all flags.  Here the ranks are sets of
    buffers on one GPU and their calls run one after another on one stream, so every flag is already set when a
    waiting merge starts (no kernel waits for a kernel that runs beside it).  Two steps through the same buffers
    with different sequence numbers; every rank's result equals the whole step and the oracle."""
    lens = [3000, 500, 37, 1, 0, 64]
    mask = np.array([[1, 0], [0, 1], [1, 1], [0, 0], [1, 0], [0, 1]], dtype=np.uint8)
    plan, ranges, ctx, layers, (Hq, Hkv, S, W, B) = _split_case(flux, layout, lens, mask, world)
    # one buffer set per layer and rank, zero-filled once
    go = [[torch.zeros((world, B, Hq, 128), dtype=torch.float32, device=DEV) for _ in range(world)] for _ in layers]
    gml = [[torch.zeros((world, B, Hq, 2), dtype=torch.float32, device=DEV) for _ in range(world)] for _ in layers]
    fl = [[torch.zeros(world, dtype=torch.int32, device=DEV) for _ in range(world)] for _ in layers]
    for step in (1, 2):
        for layer, (kt, vt, kc, vc, klog, vlog, q0) in enumerate(layers):
            q = q0 if step == 1 else synth.normal_bf16((B, Hq, 128), 44, layer, DEV)
            for r in range(world):
                kb = torch.from_numpy(ranges[r, :, 0].copy()).to(DEV)
                ke = torch.from_numpy(ranges[r, :, 1].copy()).to(DEV)
                plan.flux_attn_decode_partial_push(layer, B, q, kt, vt, ctx, kb, ke, r, go[layer], gml[layer], fl[layer], step)
            whole = plan.flux_attn_decode(layer, B, q, kt, vt, ctx)
            outs = [plan.flux_attn_combine_wait(B, go[layer][r], gml[layer][r], fl[layer][r], step) for r in range(world)]
            assert all(int(f[i]) == step for f in fl[layer] for i in range(world))
            for r in range(1, world):
                assert torch.equal(outs[r], outs[0])                   # every rank merges the same pieces in the same order
                assert torch.equal(go[layer][r], go[layer][0])
            for b, n in enumerate(lens):
                if n == 0:
                    assert torch.count_nonzero(outs[0][b]) == 0
                    continue
                ref = oracle.decode(int(mask[b, layer]), bits(q[b]), bits(klog[b]), bits(vlog[b]), n, S, W, SCALE)
                compare(outs[0][b], ref, "pushed pieces step %d layer %d b=%d" % (step, layer, b))
                compare(whole[b], ref, "single call b=%d" % b)
    assert plan.flux_plan_status() == 0


def test_waiting_merge_gives_up_when_a_piece_never_arrives(flux):
    """A flag that nothing sets: the merge's bounded wait runs out (a millisecond here), the status word reports
    it, the output is left as it was, and the plan goes on working."""
    lens = [300, 40]
    mask = np.array([[1], [0]], dtype=np.uint8)
    plan, ranges, ctx, layers, (Hq, Hkv, S, W, B) = _split_case(flux, 0, lens, mask, 2, L=1)
    kt, vt, kc, vc, klog, vlog, q = layers[0]
    go = [torch.zeros((2, B, Hq, 128), dtype=torch.float32, device=DEV) for _ in range(2)]
    gml = [torch.zeros((2, B, Hq, 2), dtype=torch.float32, device=DEV) for _ in range(2)]
    fl = [torch.zeros(2, dtype=torch.int32, device=DEV) for _ in range(2)]
    kb = torch.from_numpy(ranges[0, :, 0].copy()).to(DEV)
    ke = torch.from_numpy(ranges[0, :, 1].copy()).to(DEV)
    plan.flux_attn_decode_partial_push(0, B, q, kt, vt, ctx, kb, ke, 0, go, gml, fl, 7)      # rank 1 never pushes
    out = torch.full((B, Hq, 128), 5.0, dtype=torch.bfloat16, device=DEV)
    plan.flux_attn_combine_wait(B, go[0], gml[0], fl[0], 7, out=out, wait_cycles=2_000_000)
    with pytest.raises(flux.FluxError) as e:
        plan.flux_plan_status()
    assert e.value.code == flux.FLUX_E_DEVICE_TIMEOUT
    assert bool((out == 5.0).all())
    kb1 = torch.from_numpy(ranges[1, :, 0].copy()).to(DEV)
    ke1 = torch.from_numpy(ranges[1, :, 1].copy()).to(DEV)
    plan.flux_attn_decode_partial_push(0, B, q, kt, vt, ctx, kb1, ke1, 1, go, gml, fl, 7)
    out = plan.flux_attn_combine_wait(B, go[0], gml[0], fl[0], 7)
    for b, n in enumerate(lens):
        ref = oracle.decode(int(mask[b, 0]), bits(q[b]), bits(klog[b]), bits(vlog[b]), n, S, W, SCALE)
        compare(out[b], ref, "after the missing piece arrived b=%d" % b)
    assert plan.flux_plan_status() == 0
    with pytest.raises(flux.FluxError):
        plan.flux_attn_combine_wait(B, go[0], gml[0], fl[0], 0)                              # seq 0 is refused
