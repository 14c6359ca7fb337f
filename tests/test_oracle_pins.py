"""Pins for the fp64 CPU oracle: each check ties it to something other than itself.

The references used here are (a) hand-enumerated index lists under
``tests/golden`` (Eq. 1 / Eq. 2 with the sink + window subset), (b) closed forms
of softmax attention, (c) a second, independent evaluation written with
``math.exp`` and Python loops, (d) invariances that Eq. 1 implies.  A dropped
term, a wrong sign, an off-by-one window edge, a transposed K/V or a wrong GQA
mapping fails at least one of them.
"""
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_bits(rng, shape):
    return oracle.f64_to_bits(rng.standard_normal(shape))


def _read_sets(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            head, tail = line.split(":")
            mode, i = head.split()
            out.append((mode, int(i), [int(x) for x in tail.split()]))
    return out


# ---- index sets ---------------------------------------------------------------

@pytest.mark.parametrize("name,S,W", [("kept_sets_S2_W3.txt", 2, 3), ("kept_sets_S0_W1.txt", 0, 1)])
def test_kept_sets_match_hand_enumeration(name, S, W):
    for mode, i, want in _read_sets(name):
        got = oracle.kept(oracle.FA if mode == "FA" else oracle.SA, i, S, W)
        assert got.tolist() == want, (mode, i)


@pytest.mark.parametrize("S,W", [(64, 256), (128, 2048), (0, 5), (3, 1), (7, 7)])
def test_kept_sa_size_and_boundaries(S, W):
    N = S + W + 300
    rows = {0, max(S - 1, 0), S, max(W - 1, 0), S + W - 2, S + W - 1, S + W, S + W + 1, N - 1}
    for i in sorted(r for r in rows if r >= 0):
        idx = oracle.kept(oracle.SA, i, S, W)
        assert len(idx) == min(i + 1, S + W)
        assert np.all(np.diff(idx) > 0) and idx[-1] == i and idx[0] == (0 if (S > 0 or i < W) else i - W + 1)
        # two contiguous runs: [0, min(S, i+1)) and [max(S, i-W+1), i]
        lo = max(S, i - W + 1)
        want = list(range(0, min(S, i + 1))) + list(range(lo, i + 1))
        assert idx.tolist() == sorted(set(want))


def test_sa_equals_fa_when_sink_plus_window_covers_sequence():
    rng = np.random.default_rng(1)
    N, Hq, Hkv, D, S, W = 40, 4, 2, 8, 8, 32
    Q, K, V = (_rand_bits(rng, s) for s in [(N, Hq, D), (N, Hkv, D), (N, Hkv, D)])
    for i in range(N):
        assert oracle.kept(oracle.SA, i, S, W).tolist() == oracle.kept(oracle.FA, i, S, W).tolist()
    o_fa = oracle.prefill(oracle.FA, Q, K, V, 0, S, W, 0.3)
    o_sa = oracle.prefill(oracle.SA, Q, K, V, 0, S, W, 0.3)
    assert np.array_equal(o_fa, o_sa)          # same index list => same bits
    # and it stops being equal one position later
    assert len(oracle.kept(oracle.SA, N, S, W)) == len(oracle.kept(oracle.FA, N, S, W)) - 1


# ---- closed forms -------------------------------------------------------------

def test_two_and_three_key_closed_form():
    # q.k0 = 0, q.k1 = 1, scale = ln 3  =>  p = (1/4, 3/4)
    q = oracle.f64_to_bits(np.array([1.0, 0.0, 0.0, 0.0]))
    K = oracle.f64_to_bits(np.array([[0.0, 5.0, -2.0, 1.0], [1.0, -3.0, 0.5, 2.0], [1.0, 9.0, 9.0, 9.0]]))
    V = oracle.f64_to_bits(np.array([[4.0, 8.0, -16.0, 0.5], [-4.0, 0.0, 16.0, 1.5], [1.0, 2.0, 3.0, 4.0]]))
    o, p, m, l = oracle.attend(q, K, V, [0, 1], math.log(3.0), want_p=True)
    assert np.allclose(p, [0.25, 0.75], rtol=0, atol=1e-15)
    assert np.allclose(o, [0.25 * 4 - 0.75 * 4, 2.0, -4.0 + 12.0, 0.125 + 1.125], rtol=0, atol=1e-14)
    assert abs(m - math.log(3.0)) < 1e-15 and abs(l - (1 + 1 / 3)) < 1e-15
    # three keys, scores (0, ln2, ln2) => p = (1/5, 2/5, 2/5)
    o, p, _, _ = oracle.attend(q, K, V, [0, 1, 2], math.log(2.0), want_p=True)
    assert np.allclose(p, [0.2, 0.4, 0.4], rtol=0, atol=1e-15)
    assert np.allclose(o, 0.2 * np.array([4, 8, -16, .5]) + 0.4 * np.array([-4, 0, 16, 1.5])
                       + 0.4 * np.array([1, 2, 3, 4]), rtol=0, atol=1e-14)


def test_single_key_returns_its_value():
    rng = np.random.default_rng(2)
    Hq, Hkv, D = 6, 3, 16
    q, K, V = _rand_bits(rng, (Hq, D)), _rand_bits(rng, (1, Hkv, D)), _rand_bits(rng, (1, Hkv, D))
    for mode in (oracle.FA, oracle.SA):
        o = oracle.decode(mode, q, K, V, 1, 4, 4, 0.7)
        for h in range(Hq):
            assert np.array_equal(o[h], oracle.bits_to_f64(V[0, h // 2]))


def test_rows_sum_to_one_and_nonnegative():
    rng = np.random.default_rng(3)
    n, D = 300, 32
    q, K, V = _rand_bits(rng, (D,)), _rand_bits(rng, (n, D)), _rand_bits(rng, (n, D))
    for mode in (oracle.FA, oracle.SA):
        idx = oracle.kept(mode, n - 1, 16, 64)
        _, p, _, _ = oracle.attend(q, K, V, idx, 1 / math.sqrt(D), want_p=True)
        assert abs(p.sum() - 1.0) < 1e-12 and np.all(p >= 0)


def test_equal_keys_give_mean_and_equal_values_give_value():
    rng = np.random.default_rng(4)
    n, D, S, W = 50, 8, 4, 10
    q = _rand_bits(rng, (D,))
    k0, v0 = _rand_bits(rng, (D,)), _rand_bits(rng, (D,))
    K, V = np.tile(k0, (n, 1)), _rand_bits(rng, (n, D))
    idx = oracle.kept(oracle.SA, n - 1, S, W)
    o, _, _, _ = oracle.attend(q, K, V, idx, 0.9)
    assert np.allclose(o, oracle.bits_to_f64(V)[idx].mean(axis=0), rtol=0, atol=1e-13)
    K2, V2 = _rand_bits(rng, (n, D)), np.tile(v0, (n, 1))
    o, _, _, _ = oracle.attend(q, K2, V2, idx, 0.9)
    assert np.allclose(o, oracle.bits_to_f64(v0), rtol=0, atol=1e-13)


def test_key_shift_invariance():
    # adding one vector c to every key shifts every score of a row by scale*q.c: output unchanged
    rng = np.random.default_rng(5)
    n, D = 64, 8
    q = oracle.f64_to_bits(rng.integers(-4, 5, size=D).astype(np.float64))
    Kf = rng.integers(-8, 9, size=(n, D)).astype(np.float64)      # small integers: the shift is exact in bf16
    c = rng.integers(-8, 9, size=D).astype(np.float64)
    V = _rand_bits(rng, (n, D))
    idx = oracle.kept(oracle.FA, n - 1, 0, 1)
    o1, _, _, _ = oracle.attend(q, oracle.f64_to_bits(Kf), V, idx, 0.05)
    o2, _, _, _ = oracle.attend(q, oracle.f64_to_bits(Kf + c), V, idx, 0.05)
    assert np.allclose(o1, o2, rtol=0, atol=1e-12)


# ---- an independent second evaluation ----------------------------------------

def _brute(Qf, Kf, Vf, i, h, G, idx, scale):
    D = Qf.shape[-1]
    g = h // G
    s = []
    for j in idx:
        acc = 0.0
        for d in range(D):
            acc += Qf[i, h, d] * Kf[j, g, d]
        s.append(scale * acc)
    mx = max(s)
    e = [math.exp(x - mx) for x in s]
    z = sum(e)
    return [sum(e[t] / z * Vf[idx[t], g, d] for t in range(len(idx))) for d in range(D)]


@pytest.mark.parametrize("mode", [oracle.FA, oracle.SA])
def test_prefill_matches_python_brute_force(mode):
    rng = np.random.default_rng(6)
    N, Hq, Hkv, D, S, W = 9, 4, 2, 4, 2, 3
    Q, K, V = (_rand_bits(rng, s) for s in [(N, Hq, D), (N, Hkv, D), (N, Hkv, D)])
    Qf, Kf, Vf = (oracle.bits_to_f64(x) for x in (Q, K, V))
    golden = {(m, i): l for m, i, l in _read_sets("kept_sets_S2_W3.txt")}
    O = oracle.prefill(mode, Q, K, V, 0, S, W, 0.5)
    for i in range(N):
        name = "FA" if mode == oracle.FA else "SA"
        idx = golden.get((name, i))
        if idx is None:      # rows the fixture does not list: derive from the definition in words
            idx = [j for j in range(i + 1) if mode == oracle.FA or j < S or j >= i - W + 1]
        for h in range(Hq):
            want = _brute(Qf, Kf, Vf, i, h, Hq // Hkv, idx, 0.5)
            assert np.allclose(O[i, h], want, rtol=0, atol=1e-13), (i, h)


def test_fa_prefill_matches_dense_masked_softmax():
    # Full Attention reduces to the textbook dense causal softmax(QK^T)V
    rng = np.random.default_rng(7)
    N, H, D = 33, 3, 16
    Q, K, V = (_rand_bits(rng, (N, H, D)) for _ in range(3))
    Qf, Kf, Vf = (oracle.bits_to_f64(x) for x in (Q, K, V))
    scale = 1 / math.sqrt(D)
    O = oracle.prefill(oracle.FA, Q, K, V, 0, 0, 1, scale)
    for h in range(H):
        s = scale * Qf[:, h] @ Kf[:, h].T
        s[np.triu_indices(N, 1)] = -np.inf
        p = np.exp(s - s.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        assert np.allclose(O[:, h], p @ Vf[:, h], rtol=0, atol=1e-12)


def test_sa_prefill_matches_dense_banded_softmax():
    rng = np.random.default_rng(8)
    N, H, D, S, W = 70, 2, 8, 5, 12
    Q, K, V = (_rand_bits(rng, (N, H, D)) for _ in range(3))
    Qf, Kf, Vf = (oracle.bits_to_f64(x) for x in (Q, K, V))
    i, j = np.meshgrid(np.arange(N), np.arange(N), indexing="ij")
    allowed = (j <= i) & ((j < S) | (i - j < W))
    O = oracle.prefill(oracle.SA, Q, K, V, 0, S, W, 0.25)
    for h in range(H):
        s = np.where(allowed, 0.25 * Qf[:, h] @ Kf[:, h].T, -np.inf)
        p = np.exp(s - s.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        assert np.allclose(O[:, h], p @ Vf[:, h], rtol=0, atol=1e-12)
        assert allowed.sum(axis=1).tolist() == [min(r + 1, S + W) for r in range(N)]


# ---- structure: prefill/decode, chunking, GQA, merge, permutation -------------

@pytest.mark.parametrize("mode", [oracle.FA, oracle.SA])
def test_causal_prefix_matches_step_by_step_decode(mode):
    rng = np.random.default_rng(9)
    N, Hq, Hkv, D, S, W = 48, 4, 2, 8, 4, 9
    Q, K, V = (_rand_bits(rng, s) for s in [(N, Hq, D), (N, Hkv, D), (N, Hkv, D)])
    O = oracle.prefill(mode, Q, K, V, 0, S, W, 0.4)
    for i in range(N):
        o = oracle.decode(mode, Q[i], K, V, i + 1, S, W, 0.4)
        assert np.array_equal(o, O[i])


@pytest.mark.parametrize("mode", [oracle.FA, oracle.SA])
def test_selected_prefill_rows_address_the_same_rows_as_the_full_prefill(mode):
    """The row-subset evaluation (the one the full-size sampled checks use) against the whole-chunk
    prefill, which the brute force above pins: a chunk that starts at q_start > 0, rows out of
    order, heads repeated and out of order.  Q is indexed by (position - q_start), the output by
    the sample's own index; both slips (position used as the row, head used as the output index)
    change the result here.  Also against the pure-Python evaluation directly."""
    rng = np.random.default_rng(31)
    N, Hq, Hkv, D, S, W = 29, 6, 2, 4, 3, 5
    Q, K, V = (_rand_bits(rng, s) for s in [(N, Hq, D), (N, Hkv, D), (N, Hkv, D)])
    full = oracle.prefill(mode, Q, K, V, 0, S, W, 0.45)
    q_start = 11
    rows = np.array([28, 11, 19, 12, 28, 20, 11, 27])
    heads = np.array([5, 5, 0, 3, 1, 3, 0, 2])
    got = oracle.prefill_rows(mode, Q[q_start:], K, V, q_start, rows, heads, S, W, 0.45)
    assert got.shape == (len(rows), D)
    assert np.array_equal(got, full[rows, heads])
    assert np.array_equal(got, oracle.prefill(mode, Q[q_start:], K, V, q_start, S, W, 0.45)[rows - q_start, heads])
    Qf, Kf, Vf = (oracle.bits_to_f64(x) for x in (Q, K, V))
    for t, (i, h) in enumerate(zip(rows.tolist(), heads.tolist())):
        idx = [j for j in range(i + 1) if mode == oracle.FA or j < S or j >= i - W + 1]
        assert np.allclose(got[t], _brute(Qf, Kf, Vf, i, h, Hq // Hkv, idx, 0.45), rtol=0, atol=1e-13)
    # the rows differ from one another, so an index slip cannot hide behind equal values
    assert len({got[t].tobytes() for t in range(len(rows))}) == len({(int(i), int(h)) for i, h in zip(rows, heads)})


@pytest.mark.parametrize("mode", [oracle.FA, oracle.SA])
def test_decode_head_subset_equals_those_rows_of_the_full_decode(mode):
    """decode(heads=[...]) reads head h of q and writes sample t of the output: compare with the
    all-heads decode (pinned above through the prefill) for an unsorted list with a repeat, and
    with the pure-Python evaluation."""
    rng = np.random.default_rng(32)
    n, Hq, Hkv, D, S, W = 21, 6, 3, 4, 2, 6
    q = _rand_bits(rng, (Hq, D))
    K, V = _rand_bits(rng, (n + 3, Hkv, D)), _rand_bits(rng, (n + 3, Hkv, D))
    full = oracle.decode(mode, q, K, V, n, S, W, 0.6)
    assert full.shape == (Hq, D) and len({full[h].tobytes() for h in range(Hq)}) == Hq
    for heads in ([5, 0, 3], [3, 0, 5, 3], [4], list(range(Hq))):
        got = oracle.decode(mode, q, K, V, n, S, W, 0.6, heads=heads)
        assert got.shape == (len(heads), D)
        assert np.array_equal(got, full[heads])
    Kf, Vf = oracle.bits_to_f64(K), oracle.bits_to_f64(V)
    qf = oracle.bits_to_f64(q)[None]                 # one "row" at index 0 for the helper
    idx = [j for j in range(n) if mode == oracle.FA or j < S or j >= n - W]
    got = oracle.decode(mode, q, K, V, n, S, W, 0.6, heads=[5, 0, 3])
    for t, h in enumerate([5, 0, 3]):
        assert np.allclose(got[t], _brute(qf, Kf, Vf, 0, h, Hq // Hkv, idx, 0.6), rtol=0, atol=1e-13)


@pytest.mark.parametrize("chunk", [1, 7, 64])
def test_chunked_prefill_is_invariant(chunk):
    rng = np.random.default_rng(10)
    N, Hq, Hkv, D, S, W = 100, 2, 1, 8, 6, 20
    Q, K, V = (_rand_bits(rng, s) for s in [(N, Hq, D), (N, Hkv, D), (N, Hkv, D)])
    for mode in (oracle.FA, oracle.SA):
        whole = oracle.prefill(mode, Q, K, V, 0, S, W, 0.3)
        parts = [oracle.prefill(mode, Q[s:s + chunk], K[:s + chunk], V[:s + chunk], s, S, W, 0.3)
                 for s in range(0, N, chunk)]
        assert np.array_equal(np.concatenate(parts), whole)


def test_gqa_equals_mha_on_replicated_kv_heads():
    rng = np.random.default_rng(11)
    N, Hq, Hkv, D = 20, 6, 2, 8
    Q, K, V = (_rand_bits(rng, s) for s in [(N, Hq, D), (N, Hkv, D), (N, Hkv, D)])
    Krep, Vrep = np.repeat(K, Hq // Hkv, axis=1), np.repeat(V, Hq // Hkv, axis=1)
    for mode in (oracle.FA, oracle.SA):
        a = oracle.prefill(mode, Q, K, V, 0, 3, 5, 0.3)
        b = oracle.prefill(mode, Q, Krep, Vrep, 0, 3, 5, 0.3)
        assert np.array_equal(a, b)
    # heads 0..2 must read KV head 0 and heads 3..5 KV head 1: make KV head 1 special
    V2 = V.copy()
    V2[:, 1] = oracle.f64_to_bits(np.full((N, D), 7.0))
    o = oracle.prefill(oracle.FA, Q, K, V2, 0, 3, 5, 0.3)
    assert np.allclose(o[:, 3:], 7.0) and not np.allclose(o[:, :3], 7.0)


def test_merge_of_sink_and_window_parts_equals_sa():
    rng = np.random.default_rng(12)
    n, D, S, W = 200, 16, 8, 32
    q, K, V = _rand_bits(rng, (D,)), _rand_bits(rng, (n, D)), _rand_bits(rng, (n, D))
    idx = oracle.kept(oracle.SA, n - 1, S, W)
    o, _, m, l = oracle.attend(q, K, V, idx, 0.2)
    o1, _, m1, l1 = oracle.attend(q, K, V, idx[:S], 0.2)
    o2, _, m2, l2 = oracle.attend(q, K, V, idx[S:], 0.2)
    mm, ll, om = oracle.merge(m1, l1, o1, m2, l2, o2)
    assert np.allclose(om, o, rtol=0, atol=1e-13) and abs(mm - m) == 0 and abs(ll - l) < 1e-12 * l
    # merge is not a plain average: the pieces carry different weights
    assert not np.allclose(0.5 * (o1 + o2), o, atol=1e-6)


def test_permuting_kept_pairs_leaves_output_unchanged():
    rng = np.random.default_rng(13)
    n, D = 120, 8
    q, K, V = _rand_bits(rng, (D,)), _rand_bits(rng, (n, D)), _rand_bits(rng, (n, D))
    idx = oracle.kept(oracle.FA, n - 1, 0, 1)
    perm = rng.permutation(n)
    o1, _, _, _ = oracle.attend(q, K, V, idx, 0.3)
    o2, _, _, _ = oracle.attend(q, K[perm], V[perm], idx, 0.3)
    assert np.allclose(o1, o2, rtol=0, atol=1e-13)
    # permuting K alone does change it (K and V are not interchangeable)
    o3, _, _, _ = oracle.attend(q, K[perm], V, idx, 0.3)
    assert not np.allclose(o1, o3, atol=1e-6)


# ---- routing, sparsity ratio, retention ----------------------------------------

def test_hard_routing_and_sparsity_ratio():
    lg = np.array([[[2.0, 1.0], [0.5, 0.7], [1.0, 1.0], [-3.0, -2.0]]], dtype=np.float32)
    mask = oracle.route(lg)
    assert mask.tolist() == [[1, 0, 1, 0]]            # r_hard = 0 runs SA; a tie goes to FA
    assert oracle.msr(mask[0], 8) == 0.5
    assert oracle.msr(np.array([1, 1, 0, 1], dtype=np.uint8), 4) == 0.25
    with pytest.raises(ValueError):
        oracle.route(np.array([[[np.nan, 0.0]]], dtype=np.float32))


def test_retained_rows_and_compact_slots():
    S, W = 4, 6
    for n in range(1, 40):
        keep = oracle.retained(n, S, W)
        assert keep.tolist() == sorted(set(range(min(S, n))) | set(range(max(0, n - W), n)))
        slots = [oracle.compact_slot(int(j), S, W) for j in keep]
        assert len(set(slots)) == len(slots) and all(0 <= s < S + W for s in slots)
    # the set needed at n+1 is the set at n minus at most one row plus the new row
    for n in range(1, 40):
        a, b = set(oracle.retained(n, S, W).tolist()), set(oracle.retained(n + 1, S, W).tolist())
        assert b - a == {n} and len(a - b) <= 1


def test_compact_slot_hand_typed_values():
    """Slot rule of the compact sparse cache, typed out by hand: sink rows stay in place, the rest go
    round a ring of W rows that starts at slot S (position S -> slot S, S + W -> slot S again)."""
    table = {  # (S, W): {position: slot}
        (4, 6): {0: 0, 3: 3, 4: 4, 5: 5, 9: 9, 10: 4, 11: 5, 15: 9, 16: 4, 21: 9, 22: 4},
        (0, 3): {0: 0, 1: 1, 2: 2, 3: 0, 4: 1, 7: 1, 300: 0},
        (2, 1): {0: 0, 1: 1, 2: 2, 3: 2, 99: 2},
        (128, 4096): {127: 127, 128: 128, 4223: 4223, 4224: 128, 8319: 4223, 8320: 128, 65535: 4095, 131071: 4095},
    }
    for (S, W), rows in table.items():
        for j, want in rows.items():
            assert oracle.compact_slot(j, S, W) == want, (S, W, j)


def test_decode_byte_ratio_matches_paper_speedup():
    with open(os.path.join(GOLDEN, "decode_speedup_256k.txt")) as f:
        row = [l for l in f if l.strip() and not l.startswith("#")][0].split()
    n, omega, S, W, lo, hi = int(row[0]), float(row[1]), int(row[2]), int(row[3]), float(row[4]), float(row[5])
    rows_fa = oracle.lib().flux_oracle_kept(oracle.FA, n - 1, S, W, None)
    rows_sa = oracle.lib().flux_oracle_kept(oracle.SA, n - 1, S, W, None)
    assert rows_fa == n and rows_sa == S + W
    ratio = rows_fa / ((1 - omega) * rows_fa + omega * rows_sa)
    assert lo < ratio < hi


# ---- block-granular masks ---------------------------------------------------------

_BM_B2 = np.array([[1, 0, 0, 0], [0, 1, 0, 0], [1, 0, 1, 0], [1, 1, 0, 1]], dtype=np.uint8)


def test_block_mask_kept_sets_match_hand_enumeration():
    for _, i, want in _read_sets("kept_blocks_B2.txt"):
        assert oracle.kept_blocks(i, 2, _BM_B2).tolist() == want, i


def test_block_mask_with_unit_blocks_reproduces_sa_and_full_mask_reproduces_fa():
    """B = 1 turns the block mask into a token mask: fed with the sink + window sets it must give
    exactly the SA prefill; the lower-triangular mask at B = 4 must give exactly the FA prefill."""
    rng = np.random.default_rng(21)
    N, Hq, Hkv, D, S, W = 23, 4, 2, 8, 3, 5
    Q, K, V = (_rand_bits(rng, s) for s in [(N, Hq, D), (N, Hkv, D), (N, Hkv, D)])
    tok = np.zeros((N, N), dtype=np.uint8)
    for i in range(N):
        tok[i, oracle.kept(oracle.SA, i, S, W)] = 1
    assert np.array_equal(oracle.prefill_blocks(Q, K, V, 0, 1, tok, 0.3), oracle.prefill(oracle.SA, Q, K, V, 0, S, W, 0.3))
    nb = -(-N // 4)
    tri = np.tril(np.ones((nb, nb), dtype=np.uint8))
    assert np.array_equal(oracle.prefill_blocks(Q, K, V, 0, 4, tri, 0.3), oracle.prefill(oracle.FA, Q, K, V, 0, 0, 1, 0.3))
    # chunked evaluation and row selection address the same rows
    full = oracle.prefill_blocks(Q, K, V, 0, 4, tri, 0.3)
    part = oracle.prefill_blocks(Q[8:], K, V, 8, 4, tri, 0.3)
    assert np.array_equal(part, full[8:])
    rows, heads = np.array([0, 9, 22]), np.array([3, 0, 2])
    assert np.array_equal(oracle.prefill_blocks(Q, K, V, 0, 4, tri, 0.3, rows, heads), full[rows, heads])


def test_block_mask_prefill_matches_python_brute_force_and_empty_rows_are_zero():
    rng = np.random.default_rng(22)
    N, Hq, Hkv, D = 8, 2, 1, 4
    Q, K, V = (_rand_bits(rng, s) for s in [(N, Hq, D), (N, Hkv, D), (N, Hkv, D)])
    Qf, Kf, Vf = (oracle.bits_to_f64(x) for x in (Q, K, V))
    O = oracle.prefill_blocks(Q, K, V, 0, 2, _BM_B2, 0.7)
    for _, i, idx in _read_sets("kept_blocks_B2.txt"):
        for h in range(Hq):
            assert np.allclose(O[i, h], _brute(Qf, Kf, Vf, i, h, Hq // Hkv, idx, 0.7), rtol=0, atol=1e-13)
    bm = _BM_B2.copy()
    bm[1, 1] = 0                                     # query block 1 keeps nothing
    O2 = oracle.prefill_blocks(Q, K, V, 0, 2, bm, 0.7)
    assert not O2[2:4].any() and np.array_equal(O2[4:], O[4:])


@pytest.mark.parametrize("S,W,B", [(128, 2048, 64), (64, 256, 64), (5, 7, 4), (0, 1, 2), (130, 100, 64)])
def test_streaming_block_mask_brackets_the_token_exact_sets(S, W, B):
    """Block granularity can only round: the sink up to whole blocks, the window to the ceil(W / B)
    blocks that end with the query's own (so a row sees between W' - B + 1 and W' local positions,
    W' = W rounded up to blocks).  The kept set therefore lies between the two token-exact sets."""
    N = max(6 * B, S + W + 2 * B) + 3
    nb = -(-N // B)
    bm = oracle.streaming_block_mask(nb, nb, S, W, B)
    assert bm.shape == (nb, nb) and not np.triu(bm, 1).any() and bm.diagonal().all()
    for i in list(range(0, min(N, 3 * B + 2))) + [S + W - 1, S + W, S + W + B, N - B - 1, N - 1]:
        got = set(oracle.kept_blocks(i, B, bm).tolist())
        Wb = -(-W // B) * B
        lo = set(oracle.kept(oracle.SA, i, S, max(1, Wb - B + 1)).tolist())
        hi = set(oracle.kept(oracle.SA, i, -(-S // B) * B, Wb).tolist())
        assert lo <= got <= hi, (i, sorted(got - hi), sorted(lo - got))
    # a row far from both ends keeps ceil(S/B) sink blocks and ceil(W/B) local blocks
    assert int(bm[nb - 1].sum()) == min(nb, -(-S // B) + -(-W // B))
