"""GPU parity of the head-level comparison mode (Sec. 2.3, Appendix C.3: some heads of a layer dense,
the others sparse) against the fp64 oracle: every KV head's query group must equal the oracle's decode
in that head's mode.  Also: an all-dense / all-sparse head mask reproduces the routed layer-level
call bit for bit, and wrong layouts / bad bytes are reported."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07394_b200 import synth
from tests._util import bits, compare

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SCALE = 1.0 / np.sqrt(128.0)


@pytest.fixture(scope="module")
def flux():
    from paper_2604_07394_b200 import build, flux as f
    build.build()
    f.load()
    return f


def _caches(flux, lens, Hkv, cap, seed):
    kc, vc = [], []
    for b, n in enumerate(lens):
        k = torch.full((cap, Hkv, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
        v = torch.full_like(k, float("nan"))
        if n > 0:
            k[:n] = synth.normal_bf16((n, Hkv, 128), seed, synth.stream_id("k", 0, b), DEV)
            v[:n] = synth.normal_bf16((n, Hkv, 128), seed, synth.stream_id("v", 0, b), DEV)
        kc.append(k); vc.append(v)
    return kc, vc


@pytest.mark.parametrize("Hq,Hkv,S,W,lens", [
    (8, 2, 4, 8, [1, 12, 13, 40]),
    (28, 4, 16, 48, [64, 65, 300, 5]),
    (32, 8, 128, 256, [1000, 384, 385, 31, 0, 2500]),
    (16, 16, 32, 64, [200, 97, 4000]),
    (6, 3, 0, 1, [7, 1, 33]),
    (32, 8, 128, 2048, [70001]),                      # one long request: thousands of tiles per head
])
def test_head_level_decode_matches_oracle_per_head(flux, Hq, Hkv, S, W, lens):
    B, G = len(lens), Hq // Hkv
    cap = max(lens) + 1
    plan = flux.Plan(flux.make_config(1, Hq, Hkv, S, W, B, cap), DEV)
    rng = np.random.default_rng(Hq * 31 + Hkv)
    hm = rng.integers(0, 2, size=(B, Hkv)).astype(np.uint8)
    hm[0, :] = 0                                      # a request whose heads are all sparse
    if B > 1:
        hm[1, :] = 1                                  # ... and one whose heads are all dense
    if B > 2:
        hm[2, 0], hm[2, -1] = 1, 0                    # mixed for sure (when Hkv > 1)
    kc, vc = _caches(flux, lens, Hkv, cap, 321)
    ktab, vtab = flux.pointer_table(kc, DEV), flux.pointer_table(vc, DEV)
    ctx = torch.tensor(lens, dtype=torch.int32, device=DEV)
    q = synth.normal_bf16((B, Hq, 128), 322, 0, DEV)
    out = plan.flux_attn_decode_heads(B, q, ktab, vtab, ctx, torch.from_numpy(hm).to(DEV))
    for b, n in enumerate(lens):
        if n == 0:
            assert torch.count_nonzero(out[b]) == 0
            continue
        kb, vb = bits(kc[b][:n]), bits(vc[b][:n])
        for mode in (0, 1):
            heads = np.array([h for h in range(Hq) if hm[b, h // G] == mode], dtype=np.int64)
            if len(heads) == 0:
                continue
            ref = oracle.decode(mode, bits(q[b]), kb, vb, n, S, W, SCALE, heads=heads)
            compare(out[b][torch.from_numpy(heads).to(DEV)], ref, "head-level decode b=%d n=%d mode=%d" % (b, n, mode))
    assert plan.flux_plan_status() == 0


def test_uniform_head_masks_equal_the_layer_level_call(flux):
    Hq, Hkv, S, W, lens = 32, 8, 64, 192, [900, 257, 256, 40]
    B, cap = len(lens), 1024
    plan = flux.Plan(flux.make_config(2, Hq, Hkv, S, W, B, cap), DEV)
    plan.flux_debug_decode_kernel(flux.FLUX_DECODE_TWO_LAUNCH)      # the kernels the head-level call runs
    plan.flux_router_apply(mask=np.array([[1, 0]] * B, dtype=np.uint8))
    kc, vc = _caches(flux, lens, Hkv, cap, 55)
    ktab, vtab = flux.pointer_table(kc, DEV), flux.pointer_table(vc, DEV)
    ctx = torch.tensor(lens, dtype=torch.int32, device=DEV)
    q = synth.normal_bf16((B, Hq, 128), 56, 0, DEV)
    for layer, fill in ((0, 1), (1, 0)):
        want = plan.flux_attn_decode(layer, B, q, ktab, vtab, ctx).clone()
        hm = torch.full((B, Hkv), fill, dtype=torch.uint8, device=DEV)
        got = plan.flux_attn_decode_heads(B, q, ktab, vtab, ctx, hm)
        assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    assert plan.flux_plan_status() == 0


def test_head_level_argument_and_mask_errors(flux):
    Hq, Hkv = 8, 2
    q = synth.normal_bf16((1, Hq, 128), 1, 0, DEV)
    kc, vc = _caches(flux, [20], Hkv, 64, 9)
    ktab, vtab = flux.pointer_table(kc, DEV), flux.pointer_table(vc, DEV)
    ctx = torch.tensor([20], dtype=torch.int32, device=DEV)
    compact = flux.Plan(flux.make_config(1, Hq, Hkv, 4, 8, 1, 64, flux.FLUX_KV_COMPACT_SA), DEV)
    with pytest.raises(flux.FluxError) as e:
        compact.flux_attn_decode_heads(1, q, ktab, vtab, ctx, torch.ones((1, Hkv), dtype=torch.uint8, device=DEV))
    assert e.value.code == flux.FLUX_E_UNSUPPORTED_SHAPE
    plan = flux.Plan(flux.make_config(1, Hq, Hkv, 4, 8, 1, 64), DEV)
    with pytest.raises(flux.FluxError) as e:
        plan.flux_attn_decode_heads(1, q, ktab, vtab, ctx, np.ones((1, Hkv), dtype=np.uint8))      # host mask
    assert e.value.code == flux.FLUX_E_INVALID_ARG
    plan.flux_attn_decode_heads(1, q, ktab, vtab, ctx, torch.tensor([[1, 7]], dtype=torch.uint8, device=DEV))
    assert plan.flux_plan_status(raise_on_flag=False) == flux.FLUX_STATUS_BAD_MASK
