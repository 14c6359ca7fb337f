// Causal prefill of one routed layer on the sm_100a tensor cores (tcgen05 + TMEM + TMA).
//
// One CTA serves two query tiles at once: the same 128 query rows of two query
// heads that share a KV head (GQA) -- or, for a head left over by an odd group size (and
// for plain multi-head attention), two consecutive row tiles of one head -- so every
// K / V tile fetched by TMA feeds four MMAs.  Roles (warp-specialised, three warpgroups):
//   warps 0-3   softmax of query tile 0 (one thread per query row, TMEM lane = row)
//   warps 4-7   softmax of query tile 1
//   warp  8     TMA producer: Q once, then K_j, V_j through a ring of shared-memory slots
//   warp  9     MMA issuer: S = Q K^T (operands in shared memory), O += P V (P in TMEM)
//   warps 10-11 idle (they complete the third warpgroup, whose registers go to the softmax)
// Registers are rebalanced per warpgroup (setmaxnreg works on whole warpgroups and inside
// the CTA's own allocation): the third warpgroup shrinks to kOtherRegs, the two softmax
// warpgroups grow to kSoftmaxRegs; the host checks that the CTA's allocation covers that.
// TMEM (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each; P (bf16) overwrites the
// first 64 columns of its S.  The tensor pipe alternates between the two tiles, so the
// softmax of one tile overlaps the MMAs of the other.  Softmax is the online form in
// fp32 in the log2 domain; the running maximum is only raised when a tile exceeds it by
// more than 2^8 (the accumulator and the row sum stay consistent with the maximum in
// use, so the result is the same softmax), which makes rescaling O in TMEM rare.
// P is handed to the MMA issuer in two halves of 64 keys, so the first half of PV overlaps
// the exponentials of the second.
// An FA layer (Eq. 1) walks every KV tile up to the diagonal; an SA layer (Eq. 2 with the
// streaming subset) walks the sink tiles and the window tiles only.
//
// Every mbarrier wait is bounded: when it runs out the CTA raises
// FLUX_STATUS_WAIT_EXPIRED, stops issuing work, lets in-flight copies land, frees its
// TMEM and returns; CTAs that start after that return at once.
#include <cuda.h>

#include "flux_internal.h"
#include "flux_tc_util.h"

namespace flux {
namespace {

using namespace tc;

constexpr int BM = 128, BN = 128;
constexpr int kHalfBytes = BM * 128;              // 128 rows x 64 bf16 (one 128-byte swizzle span per row)
constexpr int kTileBytes = 2 * kHalfBytes;        // a 128 x 128 bf16 tile = two halves (d 0-63 | d 64-127)
constexpr int kKvSlots = 5;                        // K and V tiles in flight (ring of 32 KB slots)
constexpr int kThreads = 384;
constexpr int kSoftmaxThreads = 128;
constexpr int kSoftmaxRegs = 224, kOtherRegs = 56;   // per-thread register targets after rebalancing

constexpr int OFF_Q = 0;                          // Q tile 0, Q tile 1
constexpr int OFF_KV = 2 * kTileBytes;
constexpr int OFF_BAR = OFF_KV + kKvSlots * kTileBytes;
// mbarriers: Q_FULL | KV_FULL[slots] | KV_EMPTY[slots] | S_FULL[2] | P_FULL[tile][half] | O_FULL[2] |
//            Q_EMPTY   (hands the Q tiles over from one work item to the next)
constexpr int BAR_Q_FULL = 0, BAR_KV_FULL = 1, BAR_KV_EMPTY = BAR_KV_FULL + kKvSlots,
              BAR_S_FULL = BAR_KV_EMPTY + kKvSlots, BAR_P_FULL = BAR_S_FULL + 2, BAR_O_FULL = BAR_P_FULL + 4,
              BAR_Q_EMPTY = BAR_O_FULL + 2, BAR_DRAIN = BAR_Q_EMPTY + 1,   // DRAIN: only used when a CTA gives up
              kNumBars = BAR_DRAIN + 1;
static_assert(kNumBars <= 24, "barrier area");
constexpr int OFF_TMEM_PTR = OFF_BAR + 24 * 8;
constexpr int OFF_ABORT = OFF_TMEM_PTR + 4;
constexpr int kSmemBytes = OFF_BAR + 256 + 1024;  // + slack to align the base to 1024 bytes

constexpr uint32_t kTmemCols = 512;
constexpr uint32_t TM_S = 0, TM_O = 256;          // + 128 * tile

constexpr float kRescaleThreshold = 8.0f;         // log2 units

// instruction descriptor, kind::f16: D fp32, A and B bf16, M 128, N 128
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescQK = kIdescBase;               // A, B K-major
constexpr uint32_t kIdescPV = kIdescBase | (1u << 16);  // B (= V) MN-major

struct TcArgs {
    __nv_bfloat16 *out;
    const uint8_t *mask;
    int L, layer, req, Hq, G, S, W, q_start, Nq;
    int n_qt, n_kv, P, odd;      // query tiles, KV heads, head pairs per KV head, 1 if a head is left over
    int n_items;                 // work items of the launch
    float scale_log2;
    int32_t *debug;
    uint32_t *status;
    const uint8_t *bm;           // block-mask mode: uint8 [absolute query block][n_kb], blocks of 64 positions
    int n_kb;
    uint32_t *touch;             // debug bitmap of the KV positions loaded, or NULL
};

// KV tile index of the it-th tile a query tile keeps: sink tiles [0, e1), then window tiles from b2
__device__ __forceinline__ int tile_of(int it, int e1, int b2) { return it < e1 ? it : b2 + (it - e1); }

// Per-CTA constants shared by the three roles.
struct Cta {
    uint32_t sb;            // shared-window address of the 1024-byte aligned base
    uint32_t bar0;          // first mbarrier
    uint32_t tmem;          // TMEM base address
    volatile int *abort_flag;
    uint32_t *status;
    int kvh, nslots, q_end;
    int head0, head1, qt0, qt1, i00, i01;   // per query tile: query head, tile index in the chunk, first absolute position
    __device__ __forceinline__ int head(int t) const { return t ? head1 : head0; }
    __device__ __forceinline__ int qt(int t) const { return t ? qt1 : qt0; }
    __device__ __forceinline__ int i0(int t) const { return t ? i01 : i00; }
    int e1, b2, n_tiles;    // routed layers: KV tiles kept are [0, e1) and [b2, b2 + n_tiles - e1)
    bool fa;
    const uint8_t *bm;      // block-mask mode: mask, row length, last candidate KV tile
    int n_kb, last_tile;
    __device__ __forceinline__ uint32_t bar(int i) const { return bar0 + 8u * (uint32_t)i; }
    // every lane of the (converged) calling warp waits; the result is the same for all of them
    __device__ __forceinline__ bool wait(int i, uint32_t parity) const
    {
        return __all_sync(0xffffffffu, mbar_wait(bar(i), parity, abort_flag, status));
    }
};

// Work items, heaviest (latest query tiles) first.  An item is two query tiles that walk the
// same K / V tiles: the same 128 rows of two heads of a KV group, or -- for the head left
// over when the group size is odd -- two consecutive row tiles of that head (the earlier
// one simply finds its last KV tile fully masked).  Rank r = tiles counted from the end;
// ranks come in pairs (2k, 2k+1): n_kv * P head-pair items each, plus n_kv left-over items
// (tiles n_qt-1-2k and n_qt-2-2k) listed with the even rank.
__device__ __forceinline__ void decode_item(const TcArgs &a, int item, bool fa, Cta &c)
{
    const int per2 = a.n_kv * (2 * a.P + a.odd);
    const int k2 = item / per2;
    int rem = item % per2;
    int r = 2 * k2;
    bool leftover = false;
    if (rem < a.n_kv * a.P) {
    } else if (rem < a.n_kv * (a.P + a.odd)) {
        leftover = true;
        rem -= a.n_kv * a.P;
    } else {
        rem -= a.n_kv * (a.P + a.odd);
        r += 1;
    }
    const int qt = a.n_qt - 1 - r;
    if (!leftover) {
        c.kvh = rem / a.P;
        const int pi = rem % a.P;
        c.head0 = c.kvh * a.G + 2 * pi;
        c.head1 = c.head0 + 1;
        c.qt0 = c.qt1 = qt;
        c.nslots = 2;
    } else {
        c.kvh = rem;
        c.head0 = c.head1 = c.kvh * a.G + a.G - 1;
        c.qt0 = qt;
        c.qt1 = qt - 1;
        c.nslots = qt >= 1 ? 2 : 1;
    }
    c.i00 = a.q_start + c.qt0 * BM;
    c.i01 = a.q_start + c.qt1 * BM;
    const int i0_min = c.nslots == 2 ? c.i01 : c.i00;     // tile 1 is never later than tile 0
    const int i_hi = min(c.i00 + BM - 1, c.q_end - 1);
    const int e2 = i_hi / BN + 1;
    if (fa) {
        c.e1 = 0;
        c.b2 = 0;
    } else {
        c.e1 = min((a.S + BN - 1) / BN, e2);
        c.b2 = max(c.e1, max(0, i0_min - a.W + 1) / BN);
    }
    c.n_tiles = c.e1 + max(0, e2 - c.b2);
    c.last_tile = e2 - 1;
}

// The kernel is persistent: CTA b of G takes items b, 2G-1-b, 2G+b, 4G-1-b, ... (a serpentine over
// the weight-sorted list, so every CTA gets nearly the same amount of work).  Returns the k-th item
// of this CTA, or a number >= n_items when there is none.
__device__ __forceinline__ int item_of(int k)
{
    const int G = (int)gridDim.x, b = (int)blockIdx.x;
    return k * G + ((k & 1) ? G - 1 - b : b);
}

// The KV tiles of a work item, in the order every role walks them.  Called by all lanes of a
// converged warp.  Routed FA / SA layers: a plain range.  Block-mask mode: the tiles [0, last_tile]
// in which at least one kept 64 x 64 block meets the item's rows; the warp inspects 32 candidate
// tiles at a time (one per lane) and hands out the non-empty ones.  pat: for query tile t, bit
// 4 t + 2 rb + cb says that the block (row half rb, key half cb) of the 128 x 128 tile is kept.
template <bool kBlock>
struct TileWalk {
    const Cta &c;
    int it = 0, base = 0;
    uint32_t bal = 0, mypat = 0;
    __device__ __forceinline__ explicit TileWalk(const Cta &cta) : c(cta) {}
    __device__ __forceinline__ uint32_t pattern(int j) const
    {
        uint32_t pat = 0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            if (t >= c.nslots) break;
#pragma unroll
            for (int rb = 0; rb < 2; ++rb) {
                const int qb = c.i0(t) / 64 + rb;
                if (qb * 64 >= c.q_end) continue;
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) {
                    const int kb = 2 * j + cb;
                    if (kb <= qb && kb < c.n_kb && c.bm[(size_t)qb * c.n_kb + kb] != 0) pat |= 1u << (4 * t + 2 * rb + cb);
                }
            }
        }
        return pat;
    }
    __device__ __forceinline__ bool next(int &jt, uint32_t &pat)
    {
        if (!kBlock) {
            if (it >= c.n_tiles) return false;
            jt = tile_of(it++, c.e1, c.b2);
            pat = 0xffu;
            return true;
        }
        const int lane = threadIdx.x & 31;
        while (bal == 0) {
            if (base > c.last_tile) return false;
            const int j = base + lane;
            mypat = j <= c.last_tile ? pattern(j) : 0u;
            bal = __ballot_sync(0xffffffffu, mypat != 0u);
            base += 32;
        }
        const int ln = __ffs(bal) - 1;
        bal &= bal - 1;
        jt = base - 32 + ln;
        pat = __shfl_sync(0xffffffffu, mypat, ln);
        ++it;
        return true;
    }
};

// ================= TMA producer (one warp, one issuing lane) =================
template <bool kBlock>
__device__ __forceinline__ void role_load(Cta &c, const TcArgs &a, const CUtensorMap *tm_q, const CUtensorMap *tm_k,
                                          const CUtensorMap *tm_v, int &qi, int &q_armed)
{
    // qi: K / V tiles requested so far (ring position); q_armed: items whose Q tiles have been requested.  Both are
    // the caller's, so that a CTA that gives up knows which copies may still be on their way.
    for (int k = 0;; ++k) {
        const int item = item_of(k);
        if (item >= a.n_items) break;
        decode_item(a, item, c.fa, c);
        // Q of the next item may overwrite Q of this one once its last QK^T has completed
        if (k > 0 && !c.wait(BAR_Q_EMPTY, (uint32_t)((k - 1) & 1))) return;
        q_armed = k + 1;
        if (elect_one()) {
            mbar_expect_tx(c.bar(BAR_Q_FULL), (uint32_t)(c.nslots * kTileBytes));
            for (int t = 0; t < c.nslots; ++t) {
                tma_load_3d(c.sb + OFF_Q + t * kTileBytes, tm_q, c.bar(BAR_Q_FULL), 0, c.head(t), c.qt(t) * BM);
                tma_load_3d(c.sb + OFF_Q + t * kTileBytes + kHalfBytes, tm_q, c.bar(BAR_Q_FULL), 64, c.head(t), c.qt(t) * BM);
            }
        }
        TileWalk<kBlock> walk(c);
        int jt;
        uint32_t pat;
        while (walk.next(jt, pat)) {
            const int j0 = jt * BN;
            if (a.touch != nullptr) {   // debug: the positions of this tile that exist, 32 per lane 0..3
                const int lane = threadIdx.x & 31, first = j0 + 32 * lane;
                if (lane < 4 && first < c.q_end)
                    atomicOr(a.touch + (first >> 5), c.q_end - first >= 32 ? 0xffffffffu : (1u << (c.q_end - first)) - 1u);
            }
#pragma unroll
            for (int kv = 0; kv < 2; ++kv, ++qi) {
                const int slot = qi % kKvSlots, use = qi / kKvSlots;
                if (!c.wait(BAR_KV_EMPTY + slot, (uint32_t)((use & 1) ^ 1))) return;
                const uint32_t dst = c.sb + OFF_KV + slot * kTileBytes;
                const CUtensorMap *tm = kv ? tm_v : tm_k;
                if (elect_one()) {
                    mbar_expect_tx(c.bar(BAR_KV_FULL + slot), (uint32_t)kTileBytes);
                    tma_load_3d(dst, tm, c.bar(BAR_KV_FULL + slot), 0, c.kvh, j0);
                    tma_load_3d(dst + kHalfBytes, tm, c.bar(BAR_KV_FULL + slot), 64, c.kvh, j0);
                }
            }
        }
    }
}

// ================= MMA issuer (one warp, one issuing lane) =================
// Issue order per KV tile j:  PV_0[j] QK_0[j+1] PV_1[j] QK_1[j+1]; the tensor pipe runs them in
// that order, so S_t[j+1] overwrites S_t / P_t only after PV_t[j] has read P_t[j].  (One issuer for
// both tiles: two issuing warps, whose MMAs interleave instruction by instruction, ran slower.)
// Across items the same order holds (the first QK^T of an item follows the last PV of the one
// before).  The first PV of an item overwrites O_t; it waits for that item's first P_t, which the
// softmax warps of tile t publish only after their epilogue has read the previous item's O_t.
template <bool kBlock>
__device__ __forceinline__ void role_mma(Cta &c, const TcArgs &a)
{
    // S_t = Q_t K^T, then up to two commits (tcgen05.commit belongs to the issuing lane; 0 = none)
    auto qk = [&](int t, int slot, uint32_t bar_a, uint32_t bar_b) {
        const uint32_t qb = c.sb + OFF_Q + t * kTileBytes, kb = c.sb + OFF_KV + slot * kTileBytes;
        if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t off = (uint32_t)((kk >> 2) * kHalfBytes + (kk & 3) * 32);
                tc_mma_ss(c.tmem + TM_S + t * 128, smem_desc(qb + off, 16), smem_desc(kb + off, 16), kIdescQK,
                          kk > 0 ? 1u : 0u);
            }
            tc_commit(bar_a);
            if (bar_b) tc_commit(bar_b);
        }
    };
    // O_t (+)= P_t[:, 64 half ..] V[64 half ..]
    auto pv_half = [&](int t, int slot, int half, bool acc, uint32_t bar_a, uint32_t bar_b) {
        const uint32_t vb = c.sb + OFF_KV + slot * kTileBytes;
        if (elect_one()) {
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4) {
                const int kk = half * 4 + k4;
                tc_mma_ts(c.tmem + TM_O + t * 128, c.tmem + TM_S + t * 128 + kk * 8,
                          smem_desc(vb + kk * 2048, kHalfBytes), kIdescPV, (acc || kk > 0) ? 1u : 0u);
            }
            if (bar_a) tc_commit(bar_a);
            if (bar_b) tc_commit(bar_b);
        }
    };
    int qi = 0;                                      // K / V tiles consumed so far (ring position)
    int tiles[2] = {0, 0};                           // per query-tile slot: KV tiles done (barrier phases)
    for (int k = 0;; ++k) {
        const int item = item_of(k);
        if (item >= a.n_items) break;
        decode_item(a, item, c.fa, c);
        TileWalk<kBlock> walk(c);
        int jt;
        uint32_t pat;
        bool more = walk.next(jt, pat);
        if (!c.wait(BAR_Q_FULL, (uint32_t)(k & 1))) return;
        if (!more) {    // (block-mask mode) the item keeps no block at all: nothing to accumulate
            if (elect_one()) {
                for (int t = 0; t < c.nslots; ++t) tc_commit(c.bar(BAR_O_FULL + t));
                tc_commit(c.bar(BAR_Q_EMPTY));
            }
            continue;
        }
        {
            const int kslot = qi % kKvSlots, kpar = (qi / kKvSlots) & 1;
            if (!c.wait(BAR_KV_FULL + kslot, (uint32_t)kpar)) return;
            tc_fence_after();
            for (int t = 0; t < c.nslots; ++t)
                qk(t, kslot, c.bar(BAR_S_FULL + t), t == c.nslots - 1 ? c.bar(BAR_KV_EMPTY + kslot) : 0u);
            ++qi;
        }
        for (bool first = true; more; first = false) {
            const int vslot = qi % kKvSlots, vpar = (qi / kKvSlots) & 1;
            const int kslot = (qi + 1) % kKvSlots, kpar = ((qi + 1) / kKvSlots) & 1;
            more = walk.next(jt, pat);
            if (!c.wait(BAR_KV_FULL + vslot, (uint32_t)vpar)) return;
            // no QK^T of this item is left to issue once its last tile is reached: Q may be replaced
            if (!more && elect_one()) tc_commit(c.bar(BAR_Q_EMPTY));
            for (int t = 0; t < c.nslots; ++t) {
                const bool last = t == c.nslots - 1;
                if (!c.wait(BAR_P_FULL + 2 * t, (uint32_t)(tiles[t] & 1))) return;
                tc_fence_after();
                pv_half(t, vslot, 0, !first, 0u, 0u);
                if (!c.wait(BAR_P_FULL + 2 * t + 1, (uint32_t)(tiles[t] & 1))) return;
                tc_fence_after();
                // after the second half: the V slot is free once the last tile's PV is done; O is complete on the last KV tile
                pv_half(t, vslot, 1, !first, last ? c.bar(BAR_KV_EMPTY + vslot) : 0u, more ? 0u : c.bar(BAR_O_FULL + t));
                tiles[t]++;
                if (more) {
                    if (t == 0) {
                        if (!c.wait(BAR_KV_FULL + kslot, (uint32_t)kpar)) return;
                        tc_fence_after();
                    }
                    qk(t, kslot, c.bar(BAR_S_FULL + t), last ? c.bar(BAR_KV_EMPTY + kslot) : 0u);
                }
            }
            qi += more ? 2 : 1;
        }
    }
}

// ================= softmax of query tile t (one thread per query row) =================
template <bool kBlock>
__device__ __forceinline__ void role_softmax(Cta &c, const TcArgs &a, int t, int warp, int lane)
{
    const int r = (warp & 3) * 32 + lane;            // row of the tile = TMEM lane
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = c.tmem + lane_base + TM_S + t * 128;
    const uint32_t tO = c.tmem + lane_base + TM_O + t * 128;
    const int S = a.S, W = a.W;
    const float scale_log2 = a.scale_log2;
    int tiles = 0, items = 0;                        // KV tiles and items this slot has done (barrier phases)
    for (int k = 0;; ++k) {
        const int item = item_of(k);
        if (item >= a.n_items) break;
        decode_item(a, item, c.fa, c);
        if (t >= c.nslots) continue;                 // this item has a single query tile
        const int i0 = c.i0(t);                      // first absolute position of this query tile
        const int row = i0 + r;                      // absolute position of this query
        float m_used = -INFINITY;                    // running maximum in use, scaled log2 units
        float2 lsum = make_float2(0.f, 0.f);
        TileWalk<kBlock> walk(c);
        int jt;
        uint32_t pat;
        while (walk.next(jt, pat)) {
            if (!c.wait(BAR_S_FULL + t, (uint32_t)(tiles & 1))) return;
            const bool first = walk.it == 1;         // first KV tile of this item: O holds nothing yet
            ++tiles;
            tc_fence_after();
            uint32_t sr[4][32];
#pragma unroll
            for (int q = 0; q < 4; ++q) tc_ld32(tS + q * 32, sr[q]);
            tc_wait_ld();
            const int j0 = jt * BN;
            const int jmax = j0 + BN - 1;
            // this row's two block bits of the tile (block-mask mode): keys [j0, j0+64) and [j0+64, j0+128)
            const uint32_t mine = pat >> (4 * t + 2 * (r >> 6));
            const bool full = kBlock ? (jmax <= i0 && ((pat >> (4 * t)) & 0xfu) == 0xfu)
                                     : ((jmax <= i0) && (c.fa || jmax < S || j0 > i0 + BM - 1 - W));
            if (!full) {
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const int key = j0 + q * 32 + e;
                        const bool keep = kBlock ? (key <= row && ((mine >> (q >> 1)) & 1u) != 0u)
                                                 : (key <= row && (c.fa || key < S || key > row - W));
                        if (!keep) sr[q][e] = 0xff800000u;   // -inf
                    }
            }
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int e = 0; e < 32; e += 2)
                    mx[q] = fmax3(mx[q], __uint_as_float(sr[q][e]), __uint_as_float(sr[q][e + 1]));
            const float mxs = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale_log2;
            const bool need = mxs > m_used + kRescaleThreshold;
            if (__any_sync(0xffffffffu, need)) {
                const float alpha = need ? fast_exp2(m_used - mxs) : 1.0f;   // 0 when nothing was kept so far
                if (need) m_used = mxs;
                lsum.x *= alpha;
                lsum.y *= alpha;
                if (!first) {                                                // PV of the previous tile is complete
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t o[32];
                        tc_ld32(tO + q * 32, o);
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                        tc_st32(tO + q * 32, o);
                    }
                }
            }
            const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
            const float2 sc2 = make_float2(scale_log2, scale_log2), nm2 = make_float2(neg_m, neg_m);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t p[32];
                float2 acc2 = make_float2(0.f, 0.f);
#pragma unroll
                for (int qq = 0; qq < 2; ++qq)
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        float2 x = ffma2(make_float2(__uint_as_float(sr[2 * half + qq][2 * e]),
                                                     __uint_as_float(sr[2 * half + qq][2 * e + 1])), sc2, nm2);
                        x.x = fast_exp2(x.x);
                        x.y = fast_exp2(x.y);
                        if (qq == 0) lsum = fadd2(lsum, x); else acc2 = fadd2(acc2, x);
                        p[16 * qq + e] = pack_bf16(x.x, x.y);
                    }
                lsum = fadd2(lsum, acc2);
                tc_st32(tS + half * 32, p);                  // P columns [32 half, 32 half + 32) = keys [64 half, 64 half + 64)
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(c.bar(BAR_P_FULL + 2 * t + half));
            }
        }
        // ---- epilogue of the item: O / l -> bf16 -> global ----
        if (!c.wait(BAR_O_FULL + t, (uint32_t)(items & 1))) return;
        ++items;
        tc_fence_after();
        const float lrow = lsum.x + lsum.y;
        // (block-mask mode) a row whose mask keeps no key: zero output row, flagged
        const bool empty = kBlock && !(lrow > 0.f);
        if (empty && row < c.q_end) atomicOr(c.status, FLUX_STATUS_BAD_MASK);
        const float inv = empty ? 0.f : 1.0f / lrow;
        const bool valid = row < c.q_end;
        __nv_bfloat16 *dst = a.out + ((size_t)(valid ? row - a.q_start : 0) * a.Hq + c.head(t)) * kHeadDim;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint32_t o[32];
            tc_ld32(tO + q * 32, o);
            tc_wait_ld();
            if (valid) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    uint32_t w[8];
#pragma unroll
                    for (int z = 0; z < 8; ++z)
                        w[z] = empty ? 0u   // O holds nothing meaningful
                                     : pack_bf16(__uint_as_float(o[16 * e + 2 * z]) * inv, __uint_as_float(o[16 * e + 2 * z + 1]) * inv);
                    st_global_32B(dst + q * 32 + e * 16, w);
                }
            }
        }
        // The next item's first P_t is published by these same warps only after this point, and its
        // first PV (which overwrites O_t) waits for that P_t: O_t needs no hand-over barrier of its own.
    }
}

template <bool kBlock>
__global__ void __launch_bounds__(kThreads, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, TcArgs a)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    Cta c;
    c.sb = (raw + 1023u) & ~1023u;
    unsigned char *sm = smem_raw + (c.sb - raw);
    c.abort_flag = reinterpret_cast<volatile int *>(sm + OFF_ABORT);
    c.status = a.status;
    c.bar0 = c.sb + OFF_BAR;
    volatile uint32_t *tmem_ptr_smem = reinterpret_cast<volatile uint32_t *>(sm + OFF_TMEM_PTR);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // a CTA that starts after a wait has run out anywhere does nothing
    if (tid == 0) *c.abort_flag = (*reinterpret_cast<volatile uint32_t *>(a.status) & FLUX_STATUS_WAIT_EXPIRED) ? 1 : 0;
    __syncthreads();
    if (*c.abort_flag) return;

    const int bid = blockIdx.x;
    c.q_end = a.q_start + a.Nq;                           // KV rows present
    const uint8_t mode_raw = kBlock ? (uint8_t)1 : a.mask[a.req * a.L + a.layer];
    if (mode_raw > 1 && tid == 0) atomicOr(a.status, FLUX_STATUS_BAD_MASK);
    c.fa = mode_raw != 0;
    c.bm = a.bm;
    c.n_kb = a.n_kb;

    if (!kBlock && bid == 0 && tid == 0) {
        const int n = c.q_end;
        const bool two = !c.fa && n > a.S + a.W;
        int32_t *d = a.debug;
        d[0] = c.fa ? 1 : 0; d[1] = a.layer; d[2] = a.req; d[3] = n;
        d[4] = 0; d[5] = two ? a.S : n; d[6] = two ? n - a.W : 0; d[7] = two ? n : 0;
    }

    // ---- set-up: barriers, TMEM ----
    if (tid == 0) {
        mbar_init(c.bar(BAR_Q_FULL), 1);
        for (int s = 0; s < kKvSlots; ++s) {
            mbar_init(c.bar(BAR_KV_FULL + s), 1);
            mbar_init(c.bar(BAR_KV_EMPTY + s), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(c.bar(BAR_S_FULL + t), 1);
            mbar_init(c.bar(BAR_P_FULL + 2 * t), 4);       // one elected lane per softmax warp
            mbar_init(c.bar(BAR_P_FULL + 2 * t + 1), 4);
            mbar_init(c.bar(BAR_O_FULL + t), 1);
        }
        mbar_init(c.bar(BAR_Q_EMPTY), 1);
        mbar_init(c.bar(BAR_DRAIN), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(c.sb + OFF_TMEM_PTR), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    c.tmem = *tmem_ptr_smem;

    // Each warpgroup executes one setmaxnreg, all four of its warps the same one.
    int kv_requested = 0, q_requested = 0;               // the producer warp's counters (see the teardown)
    if (warp >= 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
        if (warp == 8) {
            role_load<kBlock>(c, a, &tm_q, &tm_k, &tm_v, kv_requested, q_requested);
        } else if (warp == 9) {
            role_mma<kBlock>(c, a);
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
        role_softmax<kBlock>(c, a, warp >> 2, warp, lane);
    }

    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (*c.abort_flag) {
        // A wait gave up somewhere: copies and MMAs that were already issued must land before the shared memory and
        // TMEM go away.  The producer waits for the last copy it requested into each ring slot and for the last Q
        // tiles (their barriers complete when the bytes have arrived, whoever was to consume them); the issuer commits
        // once more and waits for that commit, which follows every MMA it issued.  These waits are bounded too.
        auto drain = [&](int bar, uint32_t parity) {
            for (int i = 0; i < 200 && !mbar_try(c.bar(bar), parity); ++i) __nanosleep(1000);
        };
        if (warp == 8) {
            for (int s = 0; s < kKvSlots; ++s) {
                const int last = kv_requested - 1 - ((kv_requested - 1 - s) % kKvSlots + kKvSlots) % kKvSlots;   // latest request into slot s
                if (kv_requested > 0 && last >= 0) drain(BAR_KV_FULL + s, (uint32_t)((last / kKvSlots) & 1));
            }
            if (q_requested > 0) drain(BAR_Q_FULL, (uint32_t)((q_requested - 1) & 1));
        }
        if (warp == 9) {
            if (elect_one()) tc_commit(c.bar(BAR_DRAIN));
            drain(BAR_DRAIN, 0u);
        }
        __syncthreads();
    }
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(c.tmem), "r"(kTmemCols) : "memory");
    }
}

// One warp waits, with the bounded wait the prefill kernel uses, on an mbarrier nothing ever
// arrives at: the wait runs out after `limit` cycles, raises FLUX_STATUS_WAIT_EXPIRED and the
// kernel returns normally.  Exists so that the give-up path can be exercised without a fault.
__global__ void wait_probe_kernel(uint32_t *status, long long limit)
{
    __shared__ __align__(8) unsigned long long bar_storage;
    __shared__ int abort_flag;
    const uint32_t bar = smem_u32(&bar_storage);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    mbar_wait(bar, 0, &abort_flag, status, limit);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// [rows][heads][128] bf16 tensor viewed as (d, head, row); box = 64 columns x 1 head x 128 rows
int make_map(CUtensorMap *tm, const void *base, int heads, int rows)
{
    cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)heads, (cuuint64_t)rows};
    cuuint64_t strides[2] = {(cuuint64_t)kRowBytes, (cuuint64_t)kRowBytes * (cuuint64_t)heads};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)BM};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(FLUX_E_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return FLUX_OK;
}

}  // namespace

int prefill_tc_setup()
{
    if (!g_encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        int rc = check_cuda(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres),
                            "cudaGetDriverEntryPointByVersion(cuTensorMapEncodeTiled)");
        if (rc) return rc;
        if (qres != cudaDriverEntryPointSuccess || !fn)
            return fail(FLUX_E_CUDA, "the driver does not export cuTensorMapEncodeTiled");
        g_encode = (EncodeTiledFn)fn;
    }
    // setmaxnreg moves registers inside the CTA's own allocation (registers per thread at launch x
    // threads); a request beyond it would block for ever, so refuse to run rather than launch that.
    for (int v = 0; v < 2; ++v) {
        const void *fn = v ? (const void *)prefill_tc_kernel<true> : (const void *)prefill_tc_kernel<false>;
        cudaFuncAttributes fa;
        int rc = check_cuda(cudaFuncGetAttributes(&fa, fn), "cudaFuncGetAttributes(prefill_tc_kernel)");
        if (rc) return rc;
        if (fa.numRegs * kThreads < 2 * kSoftmaxThreads * kSoftmaxRegs + (kThreads - 2 * kSoftmaxThreads) * kOtherRegs)
            return fail(FLUX_E_CUDA, "prefill kernel was built with %d registers per thread: too few for its register rebalancing",
                        fa.numRegs);
        rc = check_cuda(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes),
                        "cudaFuncSetAttribute(prefill_tc_kernel)");
        if (rc) return rc;
    }
    return FLUX_OK;
}

int launch_wait_probe(flux_plan *p, long long limit_cycles, cudaStream_t st)
{
    wait_probe_kernel<<<1, 32, 0, st>>>((uint32_t *)((char *)p->ws + p->lay.status), limit_cycles);
    p->launches++;
    return check_cuda(cudaGetLastError(), "wait probe launch");
}

// block_mask == NULL: a routed layer (FA or SA by the cached routing bit); else block-mask mode
int launch_prefill_tc(flux_plan *p, int layer, int req, const void *q, const void *k, const void *v, int q_start,
                      int Nq, void *out, cudaStream_t st, const uint8_t *block_mask, int n_kv_blocks)
{
    const flux_config &c = p->cfg;
    char *ws = (char *)p->ws;
    CUtensorMap tq, tk, tv;
    int rc = make_map(&tq, q, c.n_q_heads, Nq);
    if (!rc) rc = make_map(&tk, k, c.n_kv_heads, q_start + Nq);
    if (!rc) rc = make_map(&tv, v, c.n_kv_heads, q_start + Nq);
    if (rc) return rc;
    TcArgs a;
    a.out = (__nv_bfloat16 *)out;
    a.mask = p->d_mask;
    a.L = c.n_layers; a.layer = layer; a.req = req; a.Hq = c.n_q_heads; a.G = p->G;
    a.S = c.sink; a.W = c.window; a.q_start = q_start; a.Nq = Nq;
    a.n_qt = (Nq + BM - 1) / BM;
    a.n_kv = c.n_kv_heads;
    a.P = p->G / 2;
    a.odd = p->G & 1;
    a.n_items = a.n_qt * a.n_kv * a.P + a.odd * a.n_kv * ((a.n_qt + 1) / 2);
    const int n_ctas = a.n_items < p->dev.n_sms ? a.n_items : p->dev.n_sms;   // persistent: one CTA per SM
    a.scale_log2 = p->scale_log2;
    a.debug = (int32_t *)(ws + p->lay.debug);
    a.status = (uint32_t *)(ws + p->lay.status);
    a.bm = block_mask;
    a.n_kb = n_kv_blocks;
    a.touch = p->touch;
    const int rec = prof_begin(p, FLUX_KERNEL_PREFILL, st);
    if (block_mask)
        prefill_tc_kernel<true><<<n_ctas, kThreads, kSmemBytes, st>>>(tq, tk, tv, a);
    else
        prefill_tc_kernel<false><<<n_ctas, kThreads, kSmemBytes, st>>>(tq, tk, tv, a);
    prof_end(p, rec, st);
    p->launches++;
    if (!block_mask) p->debug_records = 1;
    return check_cuda(cudaGetLastError(), "prefill tensor-core kernel launch");
}

}  // namespace flux
