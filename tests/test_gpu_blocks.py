"""GPU parity of the block-mask prefill (block size 64) against the fp64 oracle: random block
masks on small shapes (every row), the block-granular streaming pattern at the 32K benchmark size
(sampled rows), chunked calls, and the zero-row / status behaviour of an empty mask row."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07394_b200 import synth
from tests._util import bits, compare

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SCALE = 1.0 / np.sqrt(128.0)
B = 64


@pytest.fixture(scope="module")
def flux():
    from paper_2604_07394_b200 import build, flux as f
    build.build()
    f.load()
    return f


def _random_mask(nb, density, seed):
    rng = np.random.default_rng(seed)
    bm = (rng.random((nb, nb)) < density).astype(np.uint8)
    bm |= np.eye(nb, dtype=np.uint8)               # every query block keeps its own block
    return np.tril(bm)


@pytest.mark.parametrize("N,Hq,Hkv,density,chunks", [
    (64, 4, 2, 0.5, None),
    (130, 7, 1, 0.4, None),
    (300, 8, 2, 0.3, None),
    (520, 4, 4, 0.6, (0, 128, 448, 520)),
    (1000, 6, 2, 0.2, (0, 512, 1000)),
    (900, 3, 3, 0.15, (0, 64, 320, 900)),
])
def test_block_mask_prefill_small_shapes(flux, N, Hq, Hkv, density, chunks):
    nb = -(-N // B)
    plan = flux.Plan(flux.make_config(1, Hq, Hkv, 0, 1, 1, 1024), DEV)
    q = synth.normal_bf16((N, Hq, 128), 2000 + N, 1, DEV)
    k = synth.normal_bf16((N, Hkv, 128), 2000 + N, 2, DEV)
    v = synth.normal_bf16((N, Hkv, 128), 2000 + N, 3, DEV)
    for bm in (_random_mask(nb, density, N), oracle.streaming_block_mask(nb, nb, 64, 128, B),
               np.tril(np.ones((nb, nb), dtype=np.uint8))):
        bm_dev = torch.from_numpy(bm).to(DEV)
        ref = oracle.prefill_blocks(bits(q), bits(k), bits(v), 0, B, bm, SCALE)
        if chunks is None:
            out = plan.flux_attn_prefill_blocks(q, k, v, 0, bm_dev)
        else:
            out = torch.empty_like(q)
            for a, b in zip(chunks[:-1], chunks[1:]):
                out[a:b] = plan.flux_attn_prefill_blocks(q[a:b].contiguous(), k, v, a, bm_dev)
        compare(out, ref, "block-mask prefill N=%d" % N)
    assert plan.flux_plan_status() == 0


def test_full_block_mask_equals_fa_and_empty_row_is_flagged(flux):
    N, Hq, Hkv = 200, 4, 2
    nb = -(-N // B)
    plan = flux.Plan(flux.make_config(1, Hq, Hkv, 0, 1, 1, 1024), DEV)
    plan.flux_router_apply(mask=np.array([[1]], dtype=np.uint8))
    q = synth.normal_bf16((N, Hq, 128), 77, 1, DEV)
    k = synth.normal_bf16((N, Hkv, 128), 77, 2, DEV)
    v = synth.normal_bf16((N, Hkv, 128), 77, 3, DEV)
    tri = np.tril(np.ones((nb, nb), dtype=np.uint8))
    out = plan.flux_attn_prefill_blocks(q, k, v, 0, torch.from_numpy(tri).to(DEV))
    compare(out, oracle.prefill(oracle.FA, bits(q), bits(k), bits(v), 0, 0, 1, SCALE), "full block mask vs FA")
    assert plan.flux_plan_status() == 0
    bm = tri.copy()
    bm[1, :] = 0                                    # query block 1 keeps nothing
    out = plan.flux_attn_prefill_blocks(q, k, v, 0, torch.from_numpy(bm).to(DEV))
    ref = oracle.prefill_blocks(bits(q), bits(k), bits(v), 0, B, bm, SCALE)
    assert not ref[64:128].any() and torch.count_nonzero(out[64:128]) == 0
    compare(out[128:], ref[128:], "rows after the empty block")
    assert plan.flux_plan_status(raise_on_flag=False) == flux.FLUX_STATUS_BAD_MASK
    with pytest.raises(flux.FluxError):             # q_start must sit on a block boundary
        plan.flux_attn_prefill_blocks(q[10:], k, v, 10, torch.from_numpy(tri).to(DEV))


def test_streaming_block_mask_at_32k_sampled_rows(flux):
    """cfg2 shapes (32K tokens, 32/8 heads), sink 128 + window 2048 as 2 + 32 blocks of 64."""
    w = synth.WORKLOADS["cfg2"]
    N, Hq, Hkv, S, W = w.prompt_len, w.n_q_heads, w.n_kv_heads, w.sink, w.window
    nb = N // B
    plan = flux.Plan(flux.make_config(1, Hq, Hkv, S, W, 1, N), DEV)
    q = synth.normal_bf16((N, Hq, 128), w.seed, synth.stream_id("q"), DEV)
    k = synth.normal_bf16((N, Hkv, 128), w.seed, synth.stream_id("k"), DEV)
    v = synth.normal_bf16((N, Hkv, 128), w.seed, synth.stream_id("v"), DEV)
    bm = oracle.streaming_block_mask(nb, nb, S, W, B)
    out = plan.flux_attn_prefill_blocks(q, k, v, 0, torch.from_numpy(bm).to(DEV))
    rows = synth.sample_rows(N, S, W, 40, w.seed)
    heads = [0, 3, 4, 17, 28, 31]
    rr = np.repeat(rows, len(heads))
    hh = np.tile(np.asarray(heads, dtype=np.int64), len(rows))
    ref = oracle.prefill_blocks(bits(q), bits(k), bits(v), 0, B, bm, SCALE, rr, hh)
    compare(out[torch.from_numpy(rr).to(DEV), torch.from_numpy(hh).to(DEV)], ref, "streaming block mask at 32K")
    assert plan.flux_plan_status() == 0


@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (6, 2), (3, 3)])
def test_sparse_random_mask_with_empty_query_tiles_many_items_per_cta(flux, Hq, Hkv):
    """8192 tokens give more work items than the GPU has SMs, so CTAs of the tensor-core kernel walk
    several items each; some 128-row query tiles keep no block at all (their items issue no MMA and
    must hand the CTA's buffers on cleanly), others keep a sparse random pattern.  Even and odd group
    sizes (head pairs, left-over heads, plain multi-head attention).  Sampled rows against the oracle;
    rows of the empty tiles are zero and raise the mask flag."""
    N = 8192
    nb = N // B
    bm = _random_mask(nb, 0.06, 4242 + Hq)
    empty_tiles = [0, 5, 6, 31, 40, 62, 63]                 # first, adjacent, and the last (heaviest) tiles
    for t in empty_tiles:
        bm[2 * t:2 * t + 2, :] = 0
    bm[2 * 17, :] = 0                                       # half a tile empty: rows 2176..2239
    plan = flux.Plan(flux.make_config(1, Hq, Hkv, 0, 1, 1, N), DEV)
    q = synth.normal_bf16((N, Hq, 128), 515, 1, DEV)
    k = synth.normal_bf16((N, Hkv, 128), 515, 2, DEV)
    v = synth.normal_bf16((N, Hkv, 128), 515, 3, DEV)
    out = plan.flux_attn_prefill_blocks(q, k, v, 0, torch.from_numpy(bm).to(DEV))
    rng = np.random.default_rng(9)
    rows = np.unique(np.concatenate([rng.integers(0, N, 60), np.array([0, 127, 128, 639, 640, 895, 896, 2175, 2176, 2239, 2240,
                                                                      3967, 3968, 4095, 4096, 5119, 5120, 7935, 7936, 8191])]))
    heads = np.arange(Hq, dtype=np.int64)
    rr = np.repeat(rows, Hq)
    hh = np.tile(heads, len(rows))
    ref = oracle.prefill_blocks(bits(q), bits(k), bits(v), 0, B, bm, SCALE, rr, hh)
    got = out[torch.from_numpy(rr).to(DEV), torch.from_numpy(hh).to(DEV)]
    kept_any = np.array([bm[r // B].any() for r in rr])     # rows of an empty mask row: exact zeros on both sides
    assert not ref[~kept_any].any() and torch.count_nonzero(got[torch.from_numpy(~kept_any).to(DEV)]) == 0
    compare(got[torch.from_numpy(kept_any).to(DEV)], ref[kept_any], "sparse mask with empty tiles")
    for t in empty_tiles:
        assert torch.count_nonzero(out[128 * t:128 * t + 128]) == 0
    assert torch.count_nonzero(out[2176:2240]) == 0 and torch.count_nonzero(out[2240:2304]) > 0
    assert plan.flux_plan_status(raise_on_flag=False) == flux.FLUX_STATUS_BAD_MASK
