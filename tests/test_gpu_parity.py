"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle, element by element,
on the same seeded inputs.  Small shapes are swept in full; they span several tiles and ragged
tails.  Dispatch (mask bytes) and the KV rows each layer reads are compared bit-exactly."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07394_b200 import synth
from tests._util import bits, compact_rows_to_positions, compare, expand_ranges, logical_view

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def flux():
    from paper_2604_07394_b200 import build, flux as f
    build.build()
    f.load()
    return f


def _scale(D=128):
    return 1.0 / np.sqrt(D)


def _plan(flux, L, Hq, Hkv, S, W, B, max_ctx, layout=0, decode_kernel=None):
    cfg = flux.make_config(L, Hq, Hkv, S, W, B, max_ctx, kv_layout=layout)
    plan = flux.Plan(cfg, DEV)
    if decode_kernel is not None:
        plan.flux_debug_decode_kernel(min(decode_kernel, 2))
        plan.flux_plan_set_launch_overlap(decode_kernel == 3)
    return plan


# Both decode paths run every decode test: the two-launch pair (split-K kernel + combine pass) and the
# single-launch kernel (taken for batches of at most 32 requests when forced; larger batches fall back
# to the pair, so those cases run the pair twice); the single-launch kernel also with launch overlap on
# (schedule and first tile loads ahead of the grid-dependency wait: the calls these tests make keep the
# promise that mode asks for).
DECODE_KERNELS = pytest.mark.parametrize("dk", [1, 2, 3], ids=["two_launch", "single_launch", "single_launch_overlap"])


# ---- configuration 1 in full: prefill ---------------------------------------------------------

def test_cfg1_prefill_every_row(flux):
    w = synth.WORKLOADS["cfg1"]
    mask = synth.layer_masks(w)
    logits = synth.masks_to_logits(mask, w.seed)
    plan = _plan(flux, w.n_layers, w.n_q_heads, w.n_kv_heads, w.sink, w.window, 1, 2048)
    mask_dev = plan.flux_router_apply(logits=torch.from_numpy(logits).to(DEV))
    assert np.array_equal(mask_dev.cpu().numpy(), oracle.route(logits))
    assert mask.tolist() == [[1, 0, 1, 0]]
    N = w.prompt_len
    for layer in range(w.n_layers):
        q = synth.normal_bf16((N, w.n_q_heads, 128), w.seed, synth.stream_id("q", layer), DEV)
        k = synth.normal_bf16((N, w.n_kv_heads, 128), w.seed, synth.stream_id("k", layer), DEV)
        v = synth.normal_bf16((N, w.n_kv_heads, 128), w.seed, synth.stream_id("v", layer), DEV)
        out = plan.flux_attn_prefill(layer, 0, q, k, v, 0)
        rec = plan.flux_debug_dispatch(1)
        ref = oracle.prefill(int(mask[0, layer]), bits(q), bits(k), bits(v), 0, w.sink, w.window, _scale())
        compare(out, ref, "cfg1 prefill layer %d" % layer)
        assert rec[0, 0] == mask[0, layer] and rec[0, 1] == layer and rec[0, 3] == N
        assert expand_ranges(rec[0]) == oracle.kept(int(mask[0, layer]), N - 1, w.sink, w.window).tolist()
    assert plan.flux_plan_status() == 0


# ---- configuration 1 in full: prefill -> retain -> 16 decode steps, both cache layouts -------

@DECODE_KERNELS
@pytest.mark.parametrize("layout", [0, 1])
def test_cfg1_decode_steps(flux, layout, dk):
    w = synth.WORKLOADS["cfg1"]
    L, Hq, Hkv, S, W, N, T = w.n_layers, w.n_q_heads, w.n_kv_heads, w.sink, w.window, w.prompt_len, w.decode_steps
    mask = synth.layer_masks(w)
    plan = _plan(flux, L, Hq, Hkv, S, W, 1, N + T, layout, dk)
    plan.flux_router_apply(mask=mask)          # host mask, staged by the library
    assert np.array_equal(plan.mask.cpu().numpy(), mask)
    cap_full = N + T
    kc, vc, kfull, vfull = [], [], [], []
    for layer in range(L):
        k = synth.normal_bf16((N, Hkv, 128), w.seed, synth.stream_id("k", layer), DEV)
        v = synth.normal_bf16((N, Hkv, 128), w.seed, synth.stream_id("v", layer), DEV)
        compact = layout == 1 and mask[0, layer] == 0
        rows = S + W if compact else cap_full
        kcache = torch.zeros((rows, Hkv, 128), dtype=torch.bfloat16, device=DEV)
        vcache = torch.zeros_like(kcache)
        plan.flux_kv_retain(layer, 0, k, v, N, kcache, vcache)
        kc.append(kcache); vc.append(vcache)
        kfull.append(torch.cat([k.cpu(), torch.zeros((T, Hkv, 128), dtype=torch.bfloat16)]))
        vfull.append(torch.cat([v.cpu(), torch.zeros((T, Hkv, 128), dtype=torch.bfloat16)]))
    ktab = [flux.pointer_table([kc[l]], DEV) for l in range(L)]
    vtab = [flux.pointer_table([vc[l]], DEV) for l in range(L)]
    for step in range(T):
        n = N + step + 1
        pos = torch.tensor([n - 1], dtype=torch.int32, device=DEV)
        ctx = torch.tensor([n], dtype=torch.int32, device=DEV)
        for layer in range(L):
            mode = int(mask[0, layer])
            compact = layout == 1 and mode == 0
            qd = synth.normal_bf16((1, Hq, 128), w.seed, synth.stream_id("qdec", layer, 0, step), DEV)
            kn = synth.normal_bf16((1, Hkv, 128), w.seed, synth.stream_id("kdec", layer, 0, step), DEV)
            vn = synth.normal_bf16((1, Hkv, 128), w.seed, synth.stream_id("vdec", layer, 0, step), DEV)
            plan.flux_kv_append(layer, 1, kn, vn, ktab[layer], vtab[layer], pos)
            out = plan.flux_attn_decode(layer, 1, qd, ktab[layer], vtab[layer], ctx)
            rec = plan.flux_debug_dispatch(1)
            kfull[layer][n - 1] = kn[0].cpu(); vfull[layer][n - 1] = vn[0].cpu()
            ref = oracle.decode(mode, bits(qd[0]), bits(kfull[layer]), bits(vfull[layer]), n, S, W, _scale())
            compare(out[0], ref, "cfg1 decode step %d layer %d layout %d" % (step, layer, layout))
            # dispatch and the set of KV rows read, bit-exact
            assert rec[0, 0] == mode and rec[0, 3] == n
            rows = expand_ranges(rec[0])
            want = oracle.kept(mode, n - 1, S, W).tolist()
            if compact:
                assert compact_rows_to_positions(rows, n, S, W) == want
            else:
                assert rows == want
            if step in (0, T - 1):   # the cache itself holds what the oracle says must be retained
                kv = logical_view(kc[layer], n, S, W, compact)
                keep = oracle.retained(n, S, W) if mode == 0 else np.arange(n)
                assert torch.equal(kv[keep], kfull[layer][:n][keep])
    assert plan.flux_plan_status() == 0


# ---- small shapes: tiles, ragged tails, degenerate sink / window, GQA widths ------------------

PREFILL_CASES = [
    # N, Hq, Hkv, S, W, q_start-chunks
    (1, 4, 2, 4, 8, None),
    (63, 4, 2, 4, 8, None),
    (64, 4, 4, 0, 1, None),
    (65, 8, 2, 64, 64, None),
    (130, 7, 1, 3, 70, None),
    (300, 28, 4, 128, 100, None),
    (257, 8, 2, 0, 64, None),
    (400, 8, 8, 70, 129, (0, 100, 164, 400)),
    (520, 4, 1, 64, 256, (0, 512, 520)),
    (777, 6, 2, 130, 300, (0, 1, 129, 500, 777)),
    (1000, 3, 1, 0, 200, (0, 384, 1000)),
    (300, 4, 4, 64, 100, None),           # one query head per KV head: a CTA pairs two row tiles of a head
    (640, 5, 5, 128, 128, (0, 256, 640)),
    (129, 1, 1, 5, 9, None),
    (1000, 16, 2, 64, 256, (0, 384, 1000)),     # eight query heads per KV head: four head pairs per KV head
    (900, 12, 3, 0, 130, None),
]


@pytest.mark.parametrize("N,Hq,Hkv,S,W,chunks", PREFILL_CASES)
def test_prefill_small_shapes(flux, N, Hq, Hkv, S, W, chunks):
    plan = _plan(flux, 2, Hq, Hkv, S, W, 1, 1024)
    plan.flux_router_apply(mask=np.array([[1, 0]], dtype=np.uint8))
    seed = 1000 + N
    q = synth.normal_bf16((N, Hq, 128), seed, 1, DEV)
    k = synth.normal_bf16((N, Hkv, 128), seed, 2, DEV)
    v = synth.normal_bf16((N, Hkv, 128), seed, 3, DEV)
    for layer, mode in ((0, oracle.FA), (1, oracle.SA)):
        ref = oracle.prefill(mode, bits(q), bits(k), bits(v), 0, S, W, _scale())
        if chunks is None:
            out = plan.flux_attn_prefill(layer, 0, q, k, v, 0)
        else:
            out = torch.empty_like(q)
            for a, b in zip(chunks[:-1], chunks[1:]):
                out[a:b] = plan.flux_attn_prefill(layer, 0, q[a:b].contiguous(), k, v, a)
        compare(out, ref, "prefill N=%d mode=%d" % (N, mode))
        rec = plan.flux_debug_dispatch(1)
        assert expand_ranges(rec[0]) == oracle.kept(mode, N - 1, S, W).tolist()
    assert plan.flux_plan_status() == 0


def test_prefill_scores_rising_along_the_sequence(flux):
    """Keys whose scores grow by tens of log2 units from one KV tile to the next, so the running
    maximum has to be raised (and the accumulator rescaled) again and again in the middle of a row;
    and the mirror case, where the first keys dominate and later tiles underflow to nothing."""
    N, Hq, Hkv, S, W = 1100, 8, 2, 64, 300
    plan = _plan(flux, 2, Hq, Hkv, S, W, 1, 2048)
    plan.flux_router_apply(mask=np.array([[1, 0]], dtype=np.uint8))
    q = synth.normal_bf16((N, Hq, 128), 4242, 1, DEV).float() + 1.0
    v = synth.normal_bf16((N, Hkv, 128), 4242, 3, DEV)
    ramp = torch.linspace(0.0, 3.0, N, device=DEV)[:, None, None]
    for sign in (1.0, -1.0):
        k = (synth.normal_bf16((N, Hkv, 128), 4242, 2, DEV).float() + sign * ramp).to(torch.bfloat16)
        qb = q.to(torch.bfloat16)
        for layer, mode in ((0, oracle.FA), (1, oracle.SA)):
            out = plan.flux_attn_prefill(layer, 0, qb, k, v, 0)
            ref = oracle.prefill(mode, bits(qb), bits(k), bits(v), 0, S, W, _scale())
            compare(out, ref, "rising scores sign=%+.0f mode=%d" % (sign, mode))
    assert plan.flux_plan_status() == 0


DECODE_CASES = [
    # Hq, Hkv, S, W, context lengths (0 = inactive request), layout
    (8, 2, 4, 8, [1, 12, 13, 40], 0),
    (8, 2, 4, 8, [1, 12, 13, 40], 1),
    (28, 4, 16, 48, [64, 65, 300, 5], 0),
    (28, 4, 16, 48, [64, 65, 300, 5], 1),
    (6, 3, 0, 1, [7, 1, 33], 0),
    (16, 1, 8, 32, [500, 0, 41, 17], 1),
    (32, 8, 128, 256, [1000, 384, 385, 31], 0),
    (24, 12, 5, 20, [90, 25, 26], 1),
    (16, 16, 32, 64, [200, 97], 0),
    (28, 4, 16, 48, [20000], 0),                                   # batch 1: every CTA busy, several units each
    (28, 4, 128, 4096, [20000], 1),
    (8, 8, 64, 128, [5000, 3, 129, 128, 127, 4097, 1, 700], 1),    # a mixed batch of eight
    (8, 2, 16, 48, [70 * (b % 5) + b for b in range(32)], 0),       # the largest batch the single-launch kernel takes (incl. an inactive request)
    (32, 2, 0, 300, [2500, 2500], 0),                              # 16 query heads per KV head (two merge passes)
]


@DECODE_KERNELS
@pytest.mark.parametrize("Hq,Hkv,S,W,lens,layout", DECODE_CASES)
def test_decode_small_shapes(flux, Hq, Hkv, S, W, lens, layout, dk):
    B = len(lens)
    L = 2
    rng = np.random.default_rng(Hq * 100 + Hkv)
    mask = rng.integers(0, 2, size=(B, L)).astype(np.uint8)
    mask[0] = [1, 0]
    cap = max(lens) + 1
    plan = _plan(flux, L, Hq, Hkv, S, W, B, cap, layout, dk)
    plan.flux_router_apply(mask=torch.from_numpy(mask).to(DEV))      # device mask
    for layer in range(L):
        kc, vc, klog, vlog = [], [], [], []
        for b, n in enumerate(lens):
            compact = layout == 1 and mask[b, layer] == 0
            k = synth.normal_bf16((max(n, 1), Hkv, 128), 77, synth.stream_id("k", layer, b), DEV)
            v = synth.normal_bf16((max(n, 1), Hkv, 128), 77, synth.stream_id("v", layer, b), DEV)
            rows = S + W if compact else cap
            kcache = torch.full((rows, Hkv, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
            vcache = torch.full_like(kcache, float("nan"))
            if n > 1:   # all but the newest token come from "prefill"; the newest is appended below
                plan.flux_kv_retain(layer, b, k, v, n - 1, kcache, vcache)
            kc.append(kcache); vc.append(vcache); klog.append(k); vlog.append(v)
        ktab, vtab = flux.pointer_table(kc, DEV), flux.pointer_table(vc, DEV)
        pos = torch.tensor([n - 1 for n in lens], dtype=torch.int32, device=DEV)
        ctx = torch.tensor(lens, dtype=torch.int32, device=DEV)
        kn = torch.stack([klog[b][max(n, 1) - 1] for b, n in enumerate(lens)])
        vn = torch.stack([vlog[b][max(n, 1) - 1] for b, n in enumerate(lens)])
        plan.flux_kv_append(layer, B, kn, vn, ktab, vtab, pos)
        q = synth.normal_bf16((B, Hq, 128), 78, layer, DEV)
        out = plan.flux_attn_decode(layer, B, q, ktab, vtab, ctx)
        rec = plan.flux_debug_dispatch(B)
        for b, n in enumerate(lens):
            if n == 0:
                assert torch.count_nonzero(out[b]) == 0
                continue
            mode = int(mask[b, layer])
            ref = oracle.decode(mode, bits(q[b]), bits(klog[b]), bits(vlog[b]), n, S, W, _scale())
            compare(out[b], ref, "decode b=%d n=%d mode=%d" % (b, n, mode))
            rows = expand_ranges(rec[b])
            want = oracle.kept(mode, n - 1, S, W).tolist()
            if layout == 1 and mode == 0:
                assert compact_rows_to_positions(rows, n, S, W) == want
            else:
                assert rows == want
            assert rec[b, 0] == mode and rec[b, 2] == b
    assert plan.flux_plan_status() == 0


# ---- the KV rows the kernels read, bit for bit --------------------------------------------------

def _bits_set(words):
    w = words.cpu().numpy().astype(np.uint32)
    return np.nonzero(np.unpackbits(w.view(np.uint8), bitorder="little"))[0].tolist()


@DECODE_KERNELS
@pytest.mark.parametrize("layout", [0, 1])
def test_decode_reads_exactly_the_kept_rows(flux, layout, dk):
    """Every cache row whose K / V the decode kernel loads is recorded in a bitmap; per request the
    set must equal the oracle's kept set (mapped through the ring-slot rule for compact caches)."""
    Hq, Hkv, S, W, L = 8, 2, 16, 48, 2
    lens = [300, 64, 65, 5, 0, 1000]
    B = len(lens)
    cap = 1024
    mask = np.array([[1, 0], [0, 1], [0, 0], [0, 1], [1, 0], [0, 0]], dtype=np.uint8)
    plan = _plan(flux, L, Hq, Hkv, S, W, B, cap, layout, dk)
    plan.flux_router_apply(mask=mask)
    touched = torch.zeros((B, cap // 32), dtype=torch.int32, device=DEV)
    plan.flux_debug_touched(touched)
    for layer in range(L):
        rows = [S + W if (layout == 1 and mask[b, layer] == 0) else cap for b in range(B)]
        kc = [synth.normal_bf16((rows[b], Hkv, 128), 3, 10 * layer + b, DEV) for b in range(B)]
        vc = [synth.normal_bf16((rows[b], Hkv, 128), 4, 10 * layer + b, DEV) for b in range(B)]
        q = synth.normal_bf16((B, Hq, 128), 5, layer, DEV)
        ctx = torch.tensor(lens, dtype=torch.int32, device=DEV)
        touched.zero_()
        plan.flux_attn_decode(layer, B, q, flux.pointer_table(kc, DEV), flux.pointer_table(vc, DEV), ctx)
        torch.cuda.synchronize()
        for b, n in enumerate(lens):
            got = _bits_set(touched[b])
            if n == 0:
                assert got == []
                continue
            mode = int(mask[b, layer])
            want = oracle.kept(mode, n - 1, S, W).tolist()
            if layout == 1 and mode == 0:
                want = sorted(oracle.compact_slot(int(j), S, W) for j in want)
            assert got == want, (layer, b, n, mode)
    plan.flux_debug_touched(None)
    assert plan.flux_plan_status() == 0


def test_prefill_chunk_loads_exactly_the_tiles_its_rows_keep(flux):
    """A late chunk of a prompt: the 128-position KV tiles the tcgen05 kernel loads are exactly the
    tiles that hold a position some row of the chunk keeps (sink tiles + window tiles for SA,
    everything up to the chunk's end for FA)."""
    N, Hq, Hkv, S, W, q0 = 1000, 4, 2, 64, 200, 512
    plan = _plan(flux, 2, Hq, Hkv, S, W, 1, 1024)
    plan.flux_router_apply(mask=np.array([[1, 0]], dtype=np.uint8))
    q = synth.normal_bf16((N - q0, Hq, 128), 9, 1, DEV)
    k = synth.normal_bf16((N, Hkv, 128), 9, 2, DEV)
    v = synth.normal_bf16((N, Hkv, 128), 9, 3, DEV)
    touched = torch.zeros((1, 1024 // 32), dtype=torch.int32, device=DEV)
    plan.flux_debug_touched(touched)
    for layer, mode in ((0, oracle.FA), (1, oracle.SA)):
        touched.zero_()
        out = plan.flux_attn_prefill(layer, 0, q, k, v, q0)
        torch.cuda.synchronize()
        kept = set()
        for i in range(q0, N):
            kept.update(oracle.kept(mode, i, S, W).tolist())
        tiles = sorted({j // 128 for j in kept})
        want = [j for t in tiles for j in range(128 * t, min(N, 128 * t + 128))]
        assert _bits_set(touched[0]) == want, mode
        ref = oracle.prefill(mode, bits(q), bits(k), bits(v), q0, S, W, _scale())
        compare(out, ref, "late chunk mode %d" % mode)
    plan.flux_debug_touched(None)
    assert plan.flux_plan_status() == 0


# ---- routing and error behaviour ---------------------------------------------------------------

def test_router_inputs_and_device_flags(flux):
    plan = _plan(flux, 3, 8, 2, 4, 8, 4, 64)
    lg = np.array([[[1, 0], [0, 1], [2, 2]], [[-1, -1.5], [3, 3.5], [0, -0.0]]], dtype=np.float32)
    want = oracle.route(lg)
    assert np.array_equal(plan.flux_router_apply(logits=lg).cpu().numpy(), want)                       # host logits
    assert np.array_equal(plan.flux_router_apply(logits=torch.from_numpy(lg).to(DEV)).cpu().numpy(), want)
    assert plan.flux_plan_status() == 0
    bad = lg.copy(); bad[1, 1, 0] = np.nan
    with pytest.raises(flux.FluxError) as e:
        plan.flux_router_apply(logits=bad)
    assert e.value.code == flux.FLUX_E_INVALID_ARG
    plan.flux_router_apply(logits=torch.from_numpy(bad).to(DEV))
    assert plan.flux_plan_status(raise_on_flag=False) == flux.FLUX_STATUS_NAN_LOGIT
    assert plan.flux_plan_status() == 0                        # reading clears the word
    with pytest.raises(flux.FluxError):
        plan.flux_router_apply(mask=np.array([[1, 0, 2]], dtype=np.uint8))
    plan.flux_router_apply(mask=torch.tensor([[1, 0, 2]], dtype=torch.uint8, device=DEV))
    assert plan.flux_plan_status(raise_on_flag=False) == flux.FLUX_STATUS_BAD_MASK


def test_bounded_wait_gives_up_and_reports(flux):
    """A device-side wait that nothing satisfies runs out after its limit, sets the status bit and
    the kernel returns; the context stays usable and the next prefill is correct again."""
    plan = _plan(flux, 1, 4, 2, 8, 16, 1, 256)
    plan.flux_router_apply(mask=np.array([[1]], dtype=np.uint8))
    q = synth.normal_bf16((200, 4, 128), 31, 1, DEV)
    k = synth.normal_bf16((200, 2, 128), 31, 2, DEV)
    v = synth.normal_bf16((200, 2, 128), 31, 3, DEV)
    ref = oracle.prefill(oracle.FA, bits(q), bits(k), bits(v), 0, 8, 16, _scale())
    plan.flux_debug_wait_probe(2_000_000)                      # about a millisecond
    with pytest.raises(flux.FluxError) as e:
        plan.flux_plan_status()
    assert e.value.code == flux.FLUX_E_DEVICE_TIMEOUT
    assert plan.flux_plan_status() == 0                        # reading cleared the word
    plan.flux_debug_wait_probe(2_000_000)
    out = plan.flux_attn_prefill(0, 0, q, k, v, 0, torch.zeros_like(q))   # CTAs see the bit and do nothing
    assert plan.flux_plan_status(raise_on_flag=False) == flux.FLUX_STATUS_WAIT_EXPIRED
    assert torch.count_nonzero(out) == 0
    compare(plan.flux_attn_prefill(0, 0, q, k, v, 0), ref, "prefill after a timed-out wait")
    assert plan.flux_plan_status() == 0


def test_host_side_argument_errors_launch_nothing(flux):
    plan = _plan(flux, 2, 8, 2, 4, 8, 2, 64)
    q = torch.zeros((4, 8, 128), dtype=torch.bfloat16, device=DEV)
    k = torch.zeros((4, 2, 128), dtype=torch.bfloat16, device=DEV)
    n0 = plan.flux_launch_count()
    with pytest.raises(flux.FluxError):                         # no routing decision yet
        plan.flux_attn_prefill(0, 0, q, k, k, 0)
    plan.flux_router_apply(mask=np.array([[1, 0], [0, 1]], dtype=np.uint8))
    n1 = plan.flux_launch_count()
    assert n1 == n0 + 1
    for args in [(5, 0, q, k, k, 0), (0, 2, q, k, k, 0), (0, 0, q, k, k, 61), (0, 0, q, k, k, -1)]:
        with pytest.raises(flux.FluxError):
            plan.flux_attn_prefill(*args)
    with pytest.raises(flux.FluxError):                         # misaligned pointer
        plan.flux_attn_prefill(0, 0, q.view(-1)[1:1 + 8 * 128].view(1, 8, 128), k, k, 0)
    with pytest.raises(flux.FluxError):                         # batch beyond the routed batch
        plan.flux_attn_decode(0, 3, q, 0, 0, 0)
    assert plan.flux_launch_count() == n1
    out = plan.flux_attn_prefill(0, 0, q[:0], k, k, 0)          # Nq = 0: no-op success
    assert out.shape[0] == 0 and plan.flux_launch_count() == n1
    # a context length beyond max_context is flagged by the device and clamped
    kc = torch.zeros((64, 2, 128), dtype=torch.bfloat16, device=DEV)
    tab = flux.pointer_table([kc, kc], DEV)
    ctx = torch.tensor([65, 3], dtype=torch.int32, device=DEV)
    plan.flux_attn_decode(0, 2, torch.zeros((2, 8, 128), dtype=torch.bfloat16, device=DEV), tab, tab, ctx)
    assert plan.flux_plan_status(raise_on_flag=False) == flux.FLUX_STATUS_BAD_LENGTH


@DECODE_KERNELS
@pytest.mark.parametrize("layout", [0, 1])
def test_fused_decode_step_equals_append_then_decode(flux, layout, dk):
    """flux_attn_decode_step must leave the same caches and give the same outputs, bit for bit, as
    flux_kv_append followed by flux_attn_decode -- over several steps, so ring slots wrap."""
    Hq, Hkv, S, W, L = 8, 2, 4, 8, 2
    lens = [30, 9, 17, 0, 13]
    B = len(lens)
    plan = _plan(flux, L, Hq, Hkv, S, W, B, 64, layout, dk)
    mask = np.array([[1, 0], [0, 0], [1, 1], [0, 1], [0, 1]], dtype=np.uint8)
    plan.flux_router_apply(mask=mask)
    for layer in range(L):
        rows = [S + W if (layout == 1 and mask[b, layer] == 0) else 64 for b in range(B)]
        kc = [synth.normal_bf16((rows[b], Hkv, 128), 5, 10 * layer + b, DEV) for b in range(B)]
        vc = [synth.normal_bf16((rows[b], Hkv, 128), 6, 10 * layer + b, DEV) for b in range(B)]
        kc2 = [t.clone() for t in kc]; vc2 = [t.clone() for t in vc]
        kt, vt = flux.pointer_table(kc, DEV), flux.pointer_table(vc, DEV)
        kt2, vt2 = flux.pointer_table(kc2, DEV), flux.pointer_table(vc2, DEV)
        for step in range(12):
            n = [x + step if x > 0 else 0 for x in lens]
            ctx = torch.tensor(n, dtype=torch.int32, device=DEV)
            pos = torch.tensor([x - 1 for x in n], dtype=torch.int32, device=DEV)
            q = synth.normal_bf16((B, Hq, 128), 7, 100 * layer + step, DEV)
            kn = synth.normal_bf16((B, Hkv, 128), 8, 100 * layer + step, DEV)
            vn = synth.normal_bf16((B, Hkv, 128), 9, 100 * layer + step, DEV)
            plan.flux_kv_append(layer, B, kn, vn, kt, vt, pos)
            want = plan.flux_attn_decode(layer, B, q, kt, vt, ctx)
            got = plan.flux_attn_decode_step(layer, B, q, kn, vn, kt2, vt2, ctx)
            assert torch.equal(got, want), (layer, step)
        for b in range(B):
            assert torch.equal(kc[b], kc2[b]) and torch.equal(vc[b], vc2[b]), (layer, b)
    assert plan.flux_plan_status() == 0


@DECODE_KERNELS
@pytest.mark.parametrize("pinned", [True, False], ids=["pinned_zero_copy", "pageable_staged"])
def test_decode_host_entry_point_matches_device_entry_point(flux, pinned, dk):
    """Host buffers in, host buffers out, two layers back to back (with launch overlap the second layer's ingest
    kernel reads its host inputs while the first layer's decode launch is still running)."""
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    Hq, Hkv, S, W, B, L = 8, 2, 4, 8, 3, 2
    lens = [30, 9, 17]
    plan = _plan(flux, L, Hq, Hkv, S, W, B, 64, 0, dk)
    plan.flux_router_apply(mask=np.array([[1, 0], [0, 0], [1, 1]], dtype=np.uint8))
    kc = [synth.normal_bf16((64, Hkv, 128), 5, b, DEV) for b in range(B)]
    vc = [synth.normal_bf16((64, Hkv, 128), 6, b, DEV) for b in range(B)]
    kc2 = [t.clone() for t in kc]; vc2 = [t.clone() for t in vc]
    q = pin(synth.normal_bf16((B, Hq, 128), 7, 0, "cpu"))
    kn = pin(synth.normal_bf16((B, Hkv, 128), 7, 1, "cpu"))
    vn = pin(synth.normal_bf16((B, Hkv, 128), 7, 2, "cpu"))
    pos = torch.tensor([n - 1 for n in lens], dtype=torch.int32, device=DEV)
    ctx = torch.tensor(lens, dtype=torch.int32, device=DEV)
    out_h = [pin(torch.empty((B, Hq, 128), dtype=torch.bfloat16)) for _ in range(L)]
    kt, vt = flux.pointer_table(kc, DEV), flux.pointer_table(vc, DEV)
    for rep in range(3):                                 # the layers' calls back to back, nothing in between
        for layer in range(L):
            plan.flux_attn_decode_host(layer, B, q, kn, vn, kt, vt, pos, ctx, out_h[layer])
    torch.cuda.synchronize()
    kt2, vt2 = flux.pointer_table(kc2, DEV), flux.pointer_table(vc2, DEV)
    for layer in range(L):
        plan.flux_kv_append(layer, B, kn.to(DEV), vn.to(DEV), kt2, vt2, pos)
        out_d = plan.flux_attn_decode(layer, B, q.to(DEV), kt2, vt2, ctx)
        assert torch.equal(out_d.cpu(), out_h[layer]), layer
    assert plan.flux_plan_status() == 0


def test_decode_at_the_maximum_batch_and_group_size(flux):
    """The largest batch a plan accepts (1024 requests, ragged tiny contexts, some inactive), in both
    modes, on shared caches; and the largest group size (16 query heads per KV head).  A sample of
    the requests is checked against the oracle, inactive requests give zero rows."""
    B, Hq, Hkv, S, W = 1024, 4, 2, 4, 8
    rng = np.random.default_rng(1024)
    lens = rng.integers(0, 41, size=B).astype(np.int32)
    lens[[0, 1, 2, B - 1]] = [40, 0, 1, 33]
    mask = rng.integers(0, 2, size=(B, 1)).astype(np.uint8)
    plan = _plan(flux, 1, Hq, Hkv, S, W, B, 64)
    plan.flux_router_apply(mask=mask)
    k = synth.normal_bf16((64, Hkv, 128), 31, 1, DEV)      # every request reads the same cache (own length)
    v = synth.normal_bf16((64, Hkv, 128), 31, 2, DEV)
    ktab, vtab = flux.pointer_table([k] * B, DEV), flux.pointer_table([v] * B, DEV)
    q = synth.normal_bf16((B, Hq, 128), 32, 0, DEV)
    out = plan.flux_attn_decode(0, B, q, ktab, vtab, torch.from_numpy(lens).to(DEV))
    kb, vb = bits(k), bits(v)
    for b in list(range(0, 8)) + list(rng.integers(8, B, 40)) + [B - 1]:
        n = int(lens[b])
        if n == 0:
            assert torch.count_nonzero(out[b]) == 0
            continue
        ref = oracle.decode(int(mask[b, 0]), bits(q[b]), kb[:n], vb[:n], n, S, W, _scale())
        compare(out[b], ref, "max batch decode b=%d n=%d" % (b, n))
    assert torch.count_nonzero(out[torch.from_numpy(lens == 0).to(DEV)]) == 0
    assert plan.flux_plan_status() == 0
    with pytest.raises(flux.FluxError) as e:               # one request more than the plan was made for
        flux.Plan(flux.make_config(1, Hq, Hkv, S, W, B + 1, 64), DEV)
    assert e.value.code == flux.FLUX_E_CAPACITY

    # 16 query heads per KV head, prefill and decode
    Hq, Hkv, S, W, N = 32, 2, 16, 48, 300
    plan = _plan(flux, 2, Hq, Hkv, S, W, 1, 512)
    plan.flux_router_apply(mask=np.array([[1, 0]], dtype=np.uint8))
    qp = synth.normal_bf16((N, Hq, 128), 33, 0, DEV)
    k = synth.normal_bf16((N, Hkv, 128), 33, 1, DEV)
    v = synth.normal_bf16((N, Hkv, 128), 33, 2, DEV)
    ktab, vtab = flux.pointer_table([k], DEV), flux.pointer_table([v], DEV)
    ctx = torch.tensor([N], dtype=torch.int32, device=DEV)
    for layer, mode in ((0, oracle.FA), (1, oracle.SA)):
        compare(plan.flux_attn_prefill(layer, 0, qp, k, v, 0),
                oracle.prefill(mode, bits(qp), bits(k), bits(v), 0, S, W, _scale()), "G=16 prefill mode %d" % mode)
        compare(plan.flux_attn_decode(layer, 1, qp[N - 1:N].contiguous(), ktab, vtab, ctx)[0],
                oracle.decode(mode, bits(qp[N - 1]), bits(k), bits(v), N, S, W, _scale()), "G=16 decode mode %d" % mode)
    assert plan.flux_plan_status() == 0


def test_context_exactly_at_and_beyond_max_context(flux):
    """ctx_len == max_context is legal (the last cache row is used); max_context + 1 is clamped and
    flagged by the kernel, and the host refuses a prefill that would pass the end."""
    Hq, Hkv, S, W, cap = 8, 2, 8, 24, 257
    plan = _plan(flux, 2, Hq, Hkv, S, W, 2, cap)
    plan.flux_router_apply(mask=np.array([[1, 0], [0, 1]], dtype=np.uint8))
    k = synth.normal_bf16((cap, Hkv, 128), 41, 1, DEV)
    v = synth.normal_bf16((cap, Hkv, 128), 41, 2, DEV)
    ktab, vtab = flux.pointer_table([k, k], DEV), flux.pointer_table([v, v], DEV)
    q = synth.normal_bf16((2, Hq, 128), 42, 0, DEV)
    for layer in (0, 1):
        out = plan.flux_attn_decode(layer, 2, q, ktab, vtab, torch.tensor([cap, cap - 1], dtype=torch.int32, device=DEV))
        for b, n in ((0, cap), (1, cap - 1)):
            mode = int(plan.mask[b, layer])
            compare(out[b], oracle.decode(mode, bits(q[b]), bits(k), bits(v), n, S, W, _scale()), "ctx at capacity")
    assert plan.flux_plan_status() == 0
    plan.flux_attn_decode(0, 2, q, ktab, vtab, torch.tensor([cap + 1, 5], dtype=torch.int32, device=DEV))
    assert plan.flux_plan_status(raise_on_flag=False) == flux.FLUX_STATUS_BAD_LENGTH
    qp = synth.normal_bf16((4, Hq, 128), 43, 0, DEV)
    with pytest.raises(flux.FluxError) as e:
        plan.flux_attn_prefill(0, 0, qp, k, v, cap - 3)
    assert e.value.code == flux.FLUX_E_CAPACITY
    out = plan.flux_attn_prefill(0, 0, qp, k, v, cap - 4)      # the last four positions: fits exactly
    ref = oracle.prefill(oracle.FA, bits(qp), bits(k), bits(v), cap - 4, S, W, _scale())
    compare(out, ref, "prefill chunk ending at max_context")


@pytest.mark.parametrize("layout", [0, 1])
def test_decode_steps_replayed_as_a_graph_stay_correct(flux, layout):
    """A four-layer decode step (append + attend per layer, single-launch kernel, launch overlap on) captured
    once as a CUDA graph that also advances its own length vector, replayed 40 times: arrival counters,
    partial slots and ring slots are reused by every launch, so the last step is checked against the oracle
    in full, and the caches against the rows every step appended."""
    Hq, Hkv, S, W, L, T = 8, 2, 16, 48, 4, 40
    lens0 = [300, 40, 0]                                     # the last request stays inactive
    B = len(lens0)
    mask = np.array([[1, 0, 1, 0], [0, 0, 1, 1], [1, 1, 0, 0]], dtype=np.uint8)
    cap = max(lens0) + T + 2
    plan = _plan(flux, L, Hq, Hkv, S, W, B, cap, layout, 3)
    plan.flux_router_apply(mask=mask)
    kc, vc, klog, vlog = [], [], [], []
    for layer in range(L):
        kl, vl, kg, vg = [], [], [], []
        for b, n in enumerate(lens0):
            compact = layout == 1 and mask[b, layer] == 0
            k = synth.normal_bf16((cap, Hkv, 128), 61, 10 * layer + b, DEV)
            v = synth.normal_bf16((cap, Hkv, 128), 62, 10 * layer + b, DEV)
            kcache = torch.zeros((S + W if compact else cap, Hkv, 128), dtype=torch.bfloat16, device=DEV)
            vcache = torch.zeros_like(kcache)
            if n > 0:
                plan.flux_kv_retain(layer, b, k, v, n, kcache, vcache)
            kl.append(kcache); vl.append(vcache); kg.append(k.cpu().clone()); vg.append(v.cpu().clone())
        kc.append(kl); vc.append(vl); klog.append(kg); vlog.append(vg)
    ktab = [flux.pointer_table(kc[l], DEV) for l in range(L)]
    vtab = [flux.pointer_table(vc[l], DEV) for l in range(L)]
    q = synth.normal_bf16((L, B, Hq, 128), 63, 0, DEV)
    kn = synth.normal_bf16((L, B, Hkv, 128), 64, 0, DEV)      # the same new rows every step: what matters is where they land
    vn = synth.normal_bf16((L, B, Hkv, 128), 65, 0, DEV)
    out = torch.zeros_like(q)
    active = torch.tensor([1 if n > 0 else 0 for n in lens0], dtype=torch.int32, device=DEV)
    ctx = torch.tensor([n + 1 if n > 0 else 0 for n in lens0], dtype=torch.int32, device=DEV)   # length incl. the new token

    def step():
        for l in range(L):
            plan.flux_attn_decode_step(l, B, q[l], kn[l], vn[l], ktab[l], vtab[l], ctx, out[l])

    step()                                                   # eager once (also loads everything the capture must not)
    ctx += active
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
        ctx += active
    for _ in range(T - 2):
        graph.replay()
    torch.cuda.synchronize()
    assert plan.flux_plan_status() == 0
    # one eager step and T - 2 replays have run (capturing only records)
    steps_done = 1 + (T - 2)
    for b, n0 in enumerate(lens0):
        if n0 == 0:
            assert torch.count_nonzero(out[:, b]) == 0
            continue
        n = n0 + steps_done                                  # context length seen by the last step
        for l in range(L):
            mode = int(mask[b, l])
            kfull, vfull = klog[l][b].clone(), vlog[l][b].clone()
            kfull[n0:n] = kn[l, b].cpu(); vfull[n0:n] = vn[l, b].cpu()
            ref = oracle.decode(mode, bits(q[l, b]), bits(kfull), bits(vfull), n, S, W, _scale())
            compare(out[l, b], ref, "graph replay b=%d layer=%d mode=%d" % (b, l, mode))
            compact = layout == 1 and mode == 0
            keep = oracle.retained(n, S, W) if mode == 0 else np.arange(n)
            assert torch.equal(logical_view(kc[l][b], n, S, W, compact)[keep], kfull[:n][keep])
