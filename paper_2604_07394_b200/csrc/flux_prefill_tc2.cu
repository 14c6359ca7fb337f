// Causal prefill of one routed layer on CTA pairs (tcgen05 cta_group::2): two CTAs of a cluster
// serve the four query heads of a KV group quarter -- CTA rank c takes heads 2c and 2c + 1 of
// the quad, 128 query rows each -- and share every K / V tile: an MMA issued by the leader CTA
// (rank 0) runs on both SMs' tensor cores with M = 256 (128 rows per CTA) and takes half of
// its B operand from each CTA's shared memory.  Each CTA therefore loads and keeps only half
// of a K tile (64 of the 128 keys) and half of a V tile (64 of the 128 channels), and its
// tensor core reads 6 KB of shared memory per QK^T step instead of 8 KB, which is what bounds
// the one-CTA kernel (flux_prefill_tc.cu).  Serves routed layers (Eq. 1 / Eq. 2) whose group
// size is a multiple of four; other shapes and the block-mask mode stay on the one-CTA kernel.
//
// Per CTA the roles are those of the one-CTA kernel (warps 0-3 / 4-7 softmax of query tile
// 0 / 1, warp 8 TMA producer, warp 9 MMA issuer / TMEM allocation); only the leader's warp 9
// issues MMAs.  Barriers: the loads of both CTAs complete on the leader's Q_FULL / KV_FULL
// barriers; the leader's commits arrive on both CTAs' S_FULL / KV_EMPTY / O_FULL /
// Q_EMPTY barriers; the softmax warps of both CTAs arrive on the leader's P_FULL barriers.
// Every wait is bounded (status bit, clean exit) as in the one-CTA kernel.
#include <cuda.h>

#include "flux_internal.h"
#include "flux_tc_util.h"

namespace flux {
namespace {

using namespace tc;

constexpr int BM = 128, BN = 128;
constexpr int kHalfBytes = BM * 128;              // 128 rows x 64 bf16: half of a Q tile, or this CTA's half of a V tile
constexpr int kTileBytes = 2 * kHalfBytes;        // a 128 x 128 bf16 Q tile
constexpr int kKvBytes = 16384;                   // this CTA's half of a K tile (64 keys x 128 ch) or of a V tile (128 keys x 64 ch)
constexpr int kKvSlots = 10;                      // ring of 16 KB slots: K and V halves of five tiles
constexpr int kThreads = 384;
constexpr int kSoftmaxThreads = 128;
constexpr int kSoftmaxRegs = 224, kOtherRegs = 56;

constexpr int OFF_Q = 0;
constexpr int OFF_KV = 2 * kTileBytes;
constexpr int OFF_BAR = OFF_KV + kKvSlots * kKvBytes;
constexpr int BAR_Q_FULL = 0, BAR_KV_FULL = 1, BAR_KV_EMPTY = BAR_KV_FULL + kKvSlots,
              BAR_S_FULL = BAR_KV_EMPTY + kKvSlots, BAR_P_FULL = BAR_S_FULL + 2, BAR_O_FULL = BAR_P_FULL + 4,
              BAR_Q_EMPTY = BAR_O_FULL + 2, kNumBars = BAR_Q_EMPTY + 1;
static_assert(kNumBars <= 32, "barrier area");
constexpr int OFF_TMEM_PTR = OFF_BAR + 32 * 8;
constexpr int OFF_ABORT = OFF_TMEM_PTR + 4;
constexpr int kSmemBytes = OFF_BAR + 512 + 1024;
static_assert(kSmemBytes <= 232448, "shared memory per CTA");

constexpr uint32_t kTmemCols = 512;
constexpr uint32_t TM_S = 0, TM_O = 256;
constexpr float kRescaleThreshold = 8.0f;

// instruction descriptor, kind::f16: D fp32, A and B bf16, M 256 (128 rows per CTA), N 128
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((256u >> 4) << 24);
constexpr uint32_t kIdescQK = kIdescBase;
constexpr uint32_t kIdescPV = kIdescBase | (1u << 16);

struct PairArgs {
    __nv_bfloat16 *out;
    const uint8_t *mask;
    int L, layer, req, Hq, G, S, W, q_start, Nq;
    int n_qt, n_kv, quads;       // query tiles, KV heads, head quads per KV head
    int n_items;                 // pair items of the launch
    float scale_log2;
    int32_t *debug;
    uint32_t *status;
};

// ---- cluster-scope forms ----------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive on a barrier of another (or this) CTA of the cluster, given its cluster-window address
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status)
{
    if (mbar_try_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_cluster(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            atomicOr(status, FLUX_STATUS_WAIT_EXPIRED);
            return false;
        }
    }
}
// TMA tile load whose completion is counted on a barrier that may sit in the peer CTA
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap *tm, uint32_t cluster_bar, int c0, int c1, int c2)
{
    asm volatile("cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(dst), "l"(tm), "r"(cluster_bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// completion of all MMAs issued so far -> one arrival on the barrier at this offset in each of the two
// CTAs (two commits: this CTA's barrier and, through its cluster-window address, the peer's)
__device__ __forceinline__ void tc_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(map_to_cta(bar, 1)) : "memory");
}
__device__ __forceinline__ void tc_mma_ss_pair(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tc_mma_ts_pair(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
}

__device__ __forceinline__ int tile_of(int it, int e1, int b2) { return it < e1 ? it : b2 + (it - e1); }

struct Cta {
    uint32_t sb, bar0, lead_bar0;   // base, first barrier, the leader's first barrier (cluster-window address)
    uint32_t tmem;
    uint32_t rank;                  // 0 = leader
    volatile int *abort_flag;
    uint32_t *status;
    int kvh, head0, qt, i0, q_end;  // this CTA's two heads are head0 and head0 + 1
    int e1, b2, n_tiles;
    bool fa;
    __device__ __forceinline__ uint32_t bar(int i) const { return bar0 + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t lead_bar(int i) const { return lead_bar0 + 8u * (uint32_t)i; }
    __device__ __forceinline__ bool wait(int i, uint32_t parity) const
    {
        return __all_sync(0xffffffffu, mbar_wait(bar(i), parity, abort_flag, status));
    }
    __device__ __forceinline__ bool wait_cluster(int i, uint32_t parity) const
    {
        return __all_sync(0xffffffffu, mbar_wait_cluster(bar(i), parity, abort_flag, status));
    }
};

// Pair items, heaviest (latest query tiles) first: item = r * (n_kv * quads) + kvh * quads + quad,
// query tile n_qt - 1 - r.  Cluster g of G takes items g, 2G-1-g, 2G+g, ... (serpentine).
__device__ __forceinline__ void decode_item(const PairArgs &a, int item, Cta &c)
{
    const int per = a.n_kv * a.quads;
    const int r = item / per, rem = item % per;
    c.kvh = rem / a.quads;
    c.head0 = c.kvh * a.G + 4 * (rem % a.quads) + 2 * (int)c.rank;
    c.qt = a.n_qt - 1 - r;
    c.i0 = a.q_start + c.qt * BM;
    const int i_hi = min(c.i0 + BM - 1, c.q_end - 1);
    const int e2 = i_hi / BN + 1;
    if (c.fa) {
        c.e1 = 0;
        c.b2 = 0;
    } else {
        c.e1 = min((a.S + BN - 1) / BN, e2);
        c.b2 = max(c.e1, max(0, c.i0 - a.W + 1) / BN);
    }
    c.n_tiles = c.e1 + max(0, e2 - c.b2);
}
__device__ __forceinline__ int item_of(int k)
{
    const int G = (int)gridDim.x / 2, g = (int)blockIdx.x / 2;
    return k * G + ((k & 1) ? G - 1 - g : g);
}

// ================= TMA producer =================
// tm_k has a box of 64 keys, tm_q / tm_v one of 128 rows; all 64 channels wide.
__device__ __forceinline__ void role_load(Cta &c, const PairArgs &a, const CUtensorMap *tm_q, const CUtensorMap *tm_k,
                                          const CUtensorMap *tm_v)
{
    int qi = 0;
    for (int k = 0;; ++k) {
        const int item = item_of(k);
        if (item >= a.n_items) break;
        decode_item(a, item, c);
        if (k > 0 && !c.wait(BAR_Q_EMPTY, (uint32_t)((k - 1) & 1))) return;
        if (elect_one()) {
            // the leader's barrier counts the Q tiles of both CTAs
            if (c.rank == 0) mbar_expect_tx(c.bar(BAR_Q_FULL), (uint32_t)(4 * kTileBytes));
            for (int t = 0; t < 2; ++t) {
                tma_load_3d_pair(c.sb + OFF_Q + t * kTileBytes, tm_q, c.lead_bar(BAR_Q_FULL), 0, c.head0 + t, c.qt * BM);
                tma_load_3d_pair(c.sb + OFF_Q + t * kTileBytes + kHalfBytes, tm_q, c.lead_bar(BAR_Q_FULL), 64, c.head0 + t, c.qt * BM);
            }
        }
        for (int it = 0; it < c.n_tiles; ++it) {
            const int j0 = tile_of(it, c.e1, c.b2) * BN;
#pragma unroll
            for (int kv = 0; kv < 2; ++kv, ++qi) {
                const int slot = qi % kKvSlots, use = qi / kKvSlots;
                if (!c.wait(BAR_KV_EMPTY + slot, (uint32_t)((use & 1) ^ 1))) return;
                const uint32_t dst = c.sb + OFF_KV + slot * kKvBytes;
                if (elect_one()) {
                    if (c.rank == 0) mbar_expect_tx(c.bar(BAR_KV_FULL + slot), (uint32_t)(2 * kKvBytes));
                    if (kv == 0) {   // keys [j0 + 64 rank, + 64), both channel halves
                        tma_load_3d_pair(dst, tm_k, c.lead_bar(BAR_KV_FULL + slot), 0, c.kvh, j0 + 64 * (int)c.rank);
                        tma_load_3d_pair(dst + kKvBytes / 2, tm_k, c.lead_bar(BAR_KV_FULL + slot), 64, c.kvh, j0 + 64 * (int)c.rank);
                    } else {         // all 128 keys, channels [64 rank, + 64)
                        tma_load_3d_pair(dst, tm_v, c.lead_bar(BAR_KV_FULL + slot), 64 * (int)c.rank, c.kvh, j0);
                    }
                }
            }
        }
    }
}

// ================= MMA issuer (leader CTA only) =================
// Same issue order as the one-CTA kernel: PV_0[j] QK_0[j+1] PV_1[j] QK_1[j+1].
__device__ __forceinline__ void role_mma(Cta &c, const PairArgs &a)
{
    auto qk = [&](int t, int slot, uint32_t bar_a, uint32_t bar_b) {
        const uint32_t qb = c.sb + OFF_Q + t * kTileBytes, kb = c.sb + OFF_KV + slot * kKvBytes;
        if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t qoff = (uint32_t)((kk >> 2) * kHalfBytes + (kk & 3) * 32);
                const uint32_t koff = (uint32_t)((kk >> 2) * (kKvBytes / 2) + (kk & 3) * 32);
                tc_mma_ss_pair(c.tmem + TM_S + t * 128, smem_desc(qb + qoff, 16), smem_desc(kb + koff, 16), kIdescQK,
                               kk > 0 ? 1u : 0u);
            }
            tc_commit_pair(bar_a);
            if (bar_b) tc_commit_pair(bar_b);
        }
    };
    auto pv_half = [&](int t, int slot, int half, bool acc, uint32_t bar_a, uint32_t bar_b) {
        const uint32_t vb = c.sb + OFF_KV + slot * kKvBytes;
        if (elect_one()) {
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4) {
                const int kk = half * 4 + k4;
                tc_mma_ts_pair(c.tmem + TM_O + t * 128, c.tmem + TM_S + t * 128 + kk * 8, smem_desc(vb + kk * 2048, 16),
                               kIdescPV, (acc || kk > 0) ? 1u : 0u);
            }
            if (bar_a) tc_commit_pair(bar_a);
            if (bar_b) tc_commit_pair(bar_b);
        }
    };
    int qi = 0;
    int tiles = 0;      // KV tiles done (both query tiles advance together): phase of S_FULL / P_FULL
    for (int k = 0;; ++k) {
        const int item = item_of(k);
        if (item >= a.n_items) break;
        decode_item(a, item, c);
        if (!c.wait_cluster(BAR_Q_FULL, (uint32_t)(k & 1))) return;
        {
            const int kslot = qi % kKvSlots, kpar = (qi / kKvSlots) & 1;
            if (!c.wait_cluster(BAR_KV_FULL + kslot, (uint32_t)kpar)) return;
            tc_fence_after();
            qk(0, kslot, c.bar(BAR_S_FULL + 0), 0u);
            qk(1, kslot, c.bar(BAR_S_FULL + 1), c.bar(BAR_KV_EMPTY + kslot));
            ++qi;
        }
        for (int it = 0; it < c.n_tiles; ++it) {
            const bool more = it + 1 < c.n_tiles, first = it == 0;
            const int vslot = qi % kKvSlots, vpar = (qi / kKvSlots) & 1;
            const int kslot = (qi + 1) % kKvSlots, kpar = ((qi + 1) / kKvSlots) & 1;
            if (!c.wait_cluster(BAR_KV_FULL + vslot, (uint32_t)vpar)) return;
            if (!more && elect_one()) tc_commit_pair(c.bar(BAR_Q_EMPTY));
            for (int t = 0; t < 2; ++t) {
                const bool last = t == 1;
                if (!c.wait_cluster(BAR_P_FULL + 2 * t, (uint32_t)(tiles & 1))) return;
                tc_fence_after();
                pv_half(t, vslot, 0, !first, 0u, 0u);
                if (!c.wait_cluster(BAR_P_FULL + 2 * t + 1, (uint32_t)(tiles & 1))) return;
                tc_fence_after();
                pv_half(t, vslot, 1, !first, last ? c.bar(BAR_KV_EMPTY + vslot) : 0u, more ? 0u : c.bar(BAR_O_FULL + t));
                if (more) {
                    if (t == 0) {
                        if (!c.wait_cluster(BAR_KV_FULL + kslot, (uint32_t)kpar)) return;
                        tc_fence_after();
                    }
                    qk(t, kslot, c.bar(BAR_S_FULL + t), last ? c.bar(BAR_KV_EMPTY + kslot) : 0u);
                }
            }
            ++tiles;
            qi += more ? 2 : 1;
        }
    }
}

// ================= softmax of query tile t (one thread per query row) =================
__device__ __forceinline__ void role_softmax(Cta &c, const PairArgs &a, int t, int warp, int lane)
{
    const int r = (warp & 3) * 32 + lane;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = c.tmem + lane_base + TM_S + t * 128;
    const uint32_t tO = c.tmem + lane_base + TM_O + t * 128;
    const int S = a.S, W = a.W;
    const float scale_log2 = a.scale_log2;
    int tiles = 0, items = 0;
    for (int k = 0;; ++k) {
        const int item = item_of(k);
        if (item >= a.n_items) break;
        decode_item(a, item, c);
        const int i0 = c.i0;
        const int row = i0 + r;
        float m_used = -INFINITY;
        float2 lsum = make_float2(0.f, 0.f);
        for (int it = 0; it < c.n_tiles; ++it) {
            if (!c.wait(BAR_S_FULL + t, (uint32_t)(tiles & 1))) return;
            const bool first = it == 0;
            ++tiles;
            tc_fence_after();
            uint32_t sr[4][32];
#pragma unroll
            for (int q = 0; q < 4; ++q) tc_ld32(tS + q * 32, sr[q]);
            tc_wait_ld();
            const int j0 = tile_of(it, c.e1, c.b2) * BN;
            const int jmax = j0 + BN - 1;
            const bool full = (jmax <= i0) && (c.fa || jmax < S || j0 > i0 + BM - 1 - W);
            if (!full) {
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const int key = j0 + q * 32 + e;
                        const bool keep = key <= row && (c.fa || key < S || key > row - W);
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
                const float alpha = need ? fast_exp2(m_used - mxs) : 1.0f;
                if (need) m_used = mxs;
                lsum.x *= alpha;
                lsum.y *= alpha;
                if (!first) {
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
                tc_st32(tS + half * 32, p);
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(c.lead_bar(BAR_P_FULL + 2 * t + half));   // 8 arrivals: 4 warps of each CTA
            }
        }
        if (!c.wait(BAR_O_FULL + t, (uint32_t)(items & 1))) return;
        ++items;
        tc_fence_after();
        const float inv = 1.0f / (lsum.x + lsum.y);
        const bool valid = row < c.q_end;
        __nv_bfloat16 *dst = a.out + ((size_t)(valid ? row - a.q_start : 0) * a.Hq + c.head0 + t) * kHeadDim;
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
                        w[z] = pack_bf16(__uint_as_float(o[16 * e + 2 * z]) * inv, __uint_as_float(o[16 * e + 2 * z + 1]) * inv);
                    st_global_32B(dst + q * 32 + e * 16, w);
                }
            }
        }
    }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
prefill_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, PairArgs a)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    Cta c;
    c.sb = (raw + 1023u) & ~1023u;
    unsigned char *sm = smem_raw + (c.sb - raw);
    c.abort_flag = reinterpret_cast<volatile int *>(sm + OFF_ABORT);
    c.status = a.status;
    c.bar0 = c.sb + OFF_BAR;
    c.rank = cluster_rank();
    c.lead_bar0 = map_to_cta(c.bar0, 0);
    volatile uint32_t *tmem_ptr_smem = reinterpret_cast<volatile uint32_t *>(sm + OFF_TMEM_PTR);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // A pair that starts after a wait has run out anywhere does nothing.  Both CTAs of a pair must take
    // the same decision, so the leader reads the status word and the peer reads the leader's flag.
    if (tid == 0) *c.abort_flag = (*reinterpret_cast<volatile uint32_t *>(a.status) & FLUX_STATUS_WAIT_EXPIRED) ? 1 : 0;
    cluster_sync();
    {
        uint32_t lead_flag;
        asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(lead_flag) : "r"(map_to_cta(c.sb + OFF_ABORT, 0)) : "memory");
        cluster_sync();                      // nobody leaves (or rewrites the flag) before both have read it
        if (lead_flag) return;
        if (tid == 0) *c.abort_flag = 0;
    }

    c.q_end = a.q_start + a.Nq;
    const uint8_t mode_raw = a.mask[a.req * a.L + a.layer];
    if (mode_raw > 1 && tid == 0) atomicOr(a.status, FLUX_STATUS_BAD_MASK);
    c.fa = mode_raw != 0;
    if (blockIdx.x == 0 && tid == 0) {
        const int n = c.q_end;
        const bool two = !c.fa && n > a.S + a.W;
        int32_t *d = a.debug;
        d[0] = c.fa ? 1 : 0; d[1] = a.layer; d[2] = a.req; d[3] = n;
        d[4] = 0; d[5] = two ? a.S : n; d[6] = two ? n - a.W : 0; d[7] = two ? n : 0;
    }

    if (tid == 0) {
        mbar_init(c.bar(BAR_Q_FULL), 1);
        for (int s = 0; s < kKvSlots; ++s) {
            mbar_init(c.bar(BAR_KV_FULL + s), 1);
            mbar_init(c.bar(BAR_KV_EMPTY + s), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(c.bar(BAR_S_FULL + t), 1);
            mbar_init(c.bar(BAR_P_FULL + 2 * t), 8);       // one elected lane per softmax warp of either CTA
            mbar_init(c.bar(BAR_P_FULL + 2 * t + 1), 8);
            mbar_init(c.bar(BAR_O_FULL + t), 1);
        }
        mbar_init(c.bar(BAR_Q_EMPTY), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 9) {   // the same warp of both CTAs allocates; the columns are the same in both
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(c.sb + OFF_TMEM_PTR), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync();            // barriers of both CTAs are initialised and TMEM is there before anyone uses them
    tc_fence_after();
    c.tmem = *tmem_ptr_smem;

    if (warp >= 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
        if (warp == 8) {
            role_load(c, a, &tm_q, &tm_k, &tm_v);
        } else if (warp == 9 && c.rank == 0) {
            role_mma(c, a);
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
        role_softmax(c, a, warp >> 2, warp, lane);
    }

    // ---- teardown: neither CTA frees TMEM or leaves while its peer may still signal it ----
    tc_fence_before();
    __syncthreads();
    if (*c.abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    cluster_sync();
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(c.tmem), "r"(kTmemCols) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// [rows][heads][128] bf16 tensor viewed as (channel, head, row); box = 64 channels x 1 head x box_rows rows
int make_map(CUtensorMap *tm, const void *base, int heads, int rows, int box_rows)
{
    cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)heads, (cuuint64_t)rows};
    cuuint64_t strides[2] = {(cuuint64_t)kRowBytes, (cuuint64_t)kRowBytes * (cuuint64_t)heads};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(FLUX_E_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return FLUX_OK;
}

}  // namespace

int prefill_pair_setup()
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
    cudaFuncAttributes fa;
    int rc = check_cuda(cudaFuncGetAttributes(&fa, (const void *)prefill_pair_kernel), "cudaFuncGetAttributes(prefill_pair_kernel)");
    if (rc) return rc;
    if (fa.numRegs * kThreads < 2 * kSoftmaxThreads * kSoftmaxRegs + (kThreads - 2 * kSoftmaxThreads) * kOtherRegs)
        return fail(FLUX_E_CUDA, "pair prefill kernel was built with %d registers per thread: too few for its register rebalancing",
                    fa.numRegs);
    return check_cuda(cudaFuncSetAttribute((const void *)prefill_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes),
                      "cudaFuncSetAttribute(prefill_pair_kernel)");
}

// true if the pair kernel serves this plan's shapes (group size a multiple of four)
bool prefill_pair_supports(const flux_plan *p) { return p->G % 4 == 0; }

int launch_prefill_pair(flux_plan *p, int layer, int req, const void *q, const void *k, const void *v, int q_start,
                        int Nq, void *out, cudaStream_t st)
{
    const flux_config &c = p->cfg;
    char *ws = (char *)p->ws;
    CUtensorMap tq, tk, tv;
    int rc = make_map(&tq, q, c.n_q_heads, Nq, BM);
    if (!rc) rc = make_map(&tk, k, c.n_kv_heads, q_start + Nq, 64);
    if (!rc) rc = make_map(&tv, v, c.n_kv_heads, q_start + Nq, BN);
    if (rc) return rc;
    PairArgs a;
    a.out = (__nv_bfloat16 *)out;
    a.mask = p->d_mask;
    a.L = c.n_layers; a.layer = layer; a.req = req; a.Hq = c.n_q_heads; a.G = p->G;
    a.S = c.sink; a.W = c.window; a.q_start = q_start; a.Nq = Nq;
    a.n_qt = (Nq + BM - 1) / BM;
    a.n_kv = c.n_kv_heads;
    a.quads = p->G / 4;
    a.n_items = a.n_qt * a.n_kv * a.quads;
    a.scale_log2 = p->scale_log2;
    a.debug = (int32_t *)(ws + p->lay.debug);
    a.status = (uint32_t *)(ws + p->lay.status);
    const int max_pairs = p->dev.n_sms / 2;
    const int n_pairs = a.n_items < max_pairs ? a.n_items : max_pairs;
    const int rec = prof_begin(p, FLUX_KERNEL_PREFILL, st);
    prefill_pair_kernel<<<2 * n_pairs, kThreads, kSmemBytes, st>>>(tq, tk, tv, a);
    prof_end(p, rec, st);
    p->launches++;
    p->debug_records = 1;
    return check_cuda(cudaGetLastError(), "pair prefill kernel launch");
}

}  // namespace flux
