"""The workspace-free decode entry point against the regular one.

``flux_attn_decode_noalloc`` exists for callers that cannot allocate device memory (a plug-in
inside a program that owns all of it, a loop that must avoid the synchronisation an allocation
may cause); its scratch is a fixed array inside the library.  The test calls it through the
C ABI twice in a row, with different inputs, and compares each result with what
``flux_attn_decode`` (workspace supplied by the caller) gives for the same inputs.  It lives
in a file that sorts last so that a failure here cannot hide the other tests' results."""
import numpy as np
import pytest
import torch

from paper_2604_07394_b200 import synth
from tests._util import compare

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_noalloc_decode_matches_workspace_decode_twice_in_a_row():
    from paper_2604_07394_b200 import build, flux
    build.build()
    flux.load()
    L, Hq, Hkv, S, W = 2, 28, 4, 16, 48
    lens = [300, 64, 65, 5, 1]
    B = len(lens)
    mask = np.array([[1, 0], [0, 1], [0, 0], [1, 1], [0, 1]], dtype=np.uint8)
    cfg = flux.make_config(L, Hq, Hkv, S, W, B, 512, kv_layout=flux.FLUX_KV_FULL)
    plan = flux.Plan(cfg, DEV)
    mask_dev = plan.flux_router_apply(mask=mask)
    kc = [synth.normal_bf16((512, Hkv, 128), 91, b, DEV) for b in range(B)]
    vc = [synth.normal_bf16((512, Hkv, 128), 92, b, DEV) for b in range(B)]
    ktab, vtab = flux.pointer_table(kc, DEV), flux.pointer_table(vc, DEV)
    ctx = torch.tensor(lens, dtype=torch.int32, device=DEV)
    status = torch.full((1,), 77, dtype=torch.int32, device=DEV)
    for call, layer in enumerate((0, 1)):
        q = synth.normal_bf16((B, Hq, 128), 93, layer, DEV)
        want = plan.flux_attn_decode(layer, B, q, ktab, vtab, ctx)
        out = torch.zeros_like(q)
        flux.flux_attn_decode_noalloc(cfg, layer, B, mask_dev, q, ktab, vtab, ctx, out, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        compare(out, want.float().cpu().numpy().astype(np.float64), "noalloc call %d" % call)
    assert plan.flux_plan_status() == 0
    # sizes beyond the built-in scratch are refused with a clear message, nothing is launched
    big = flux.make_config(L, Hq, Hkv, S, W, 65, 512)
    with pytest.raises(flux.FluxError) as e:
        flux.flux_attn_decode_noalloc(big, 0, 65, mask_dev, q, ktab, vtab, ctx, out, None)
    assert e.value.code == flux.FLUX_E_CAPACITY and "64" in str(e.value)
    wide = flux.make_config(L, 32, 2, S, W, B, 512)      # 16 query heads per KV head
    with pytest.raises(flux.FluxError) as e:
        flux.flux_attn_decode_noalloc(wide, 0, B, mask_dev, q, ktab, vtab, ctx, out, None)
    assert e.value.code == flux.FLUX_E_CAPACITY
