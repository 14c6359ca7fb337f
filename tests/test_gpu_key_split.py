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
