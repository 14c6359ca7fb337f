// Single-launch split-K decode for small batches (sm_100a).
//
// At batch 1 (the latency protocol of Appendix C.3) a sparse layer reads a few megabytes: the
// launch is bound by fixed costs, not by bandwidth, and a second launch that merges the split-K
// partials costs as much as the attention itself.  This kernel does the whole layer in one launch:
//
//  * work is split by (request, KV head, 128-token tile): a CTA streams one KV head's 256-byte
//    row pieces, its eight warps taking 16 tokens each, so a CTA produces partials for the G query
//    heads of one KV head only (a quarter or an eighth of what a whole-row CTA would write);
//  * when a CTA leaves a (request, KV head) segment its eight warps merge their flash-attention
//    states through shared memory into one partial (O, m, l) per query head;
//  * the CTA then takes a ticket on the segment's arrival counter; the CTA that draws the last
//    ticket merges the segment's partials (Eq. 1 / Eq. 2 are sums over disjoint key sets, which
//    merge by rescaling with 2^(m_p - m)) and writes the bf16 output rows.  Nobody waits: every
//    CTA but the last simply leaves.
//
// The launch is issued with programmatic stream serialisation and releases its dependents at once, so
// the next launch of this kind is set up while this one drains.  By default the kernel waits for the
// previous launch (griddepcontrol.wait) before it touches global memory.  In overlap mode
// (flux_plan_set_launch_overlap) it first reads what the caller has promised the previous launch
// does not write -- lengths, routing mask, pointer tables and every cache row but the newest -- builds
// its schedule and starts its first tile loads, and only then waits; the newest row, the query rows
// and everything the kernel writes come after the wait.
#include "flux_decode_common.h"

namespace flux {
namespace {

constexpr int kFuCtaTok = kDecWarps * kDecTile;   // tokens of one KV head per unit
constexpr int kFuRows = 8;                        // query heads merged per pass (G <= 16: two passes)
constexpr int kFuRowStride = kHeadDim + 4;        // floats; the pad spreads the rows over the banks
constexpr int kFuStageBytes = kDecWarps * kDecStages * kDecStageBytes;
constexpr int kFuMergeOBytes = kDecWarps * kFuRows * kFuRowStride * (int)sizeof(float);
constexpr int kFuMergeMlBytes = kDecWarps * kFuRows * 2 * (int)sizeof(float);
constexpr int kFuSmemBytes = kFuStageBytes + kFuMergeOBytes + kFuMergeMlBytes;
// partial rows (512 bytes of O and 8 bytes of (m, l) each) the idle stage memory takes for the last CTA's merge
constexpr int kFuStagedRows = kFuStageBytes / (kHeadDim * 4 + 8);

struct FuIt {
    int u;      // global unit index
    int b;      // request
    int head;   // KV head
    int x;      // 128-token tile inside the request
    int tiles;  // tiles of request b
    int base;   // first unit of request b
};

// Row `row` of the merge buffers, summed over the eight warps' entries with the split-K weights.
// Returns the merged (m, l) and this lane's four output channels (unnormalised).
__device__ __forceinline__ float4 fu_merge_row(const float *mo, const float *mml, int row, int lane, float &m_out,
                                               float &l_out)
{
    float mp[kDecWarps], lp[kDecWarps];
    float m = kNegBig;
#pragma unroll
    for (int s = 0; s < kDecWarps; ++s) {
        const float2 ml = *reinterpret_cast<const float2 *>(mml + (s * kFuRows + row) * 2);
        mp[s] = ml.x;
        lp[s] = ml.y;
        m = fmaxf(m, ml.x);
    }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
#pragma unroll
    for (int s = 0; s < kDecWarps; ++s) {
        const float w = fast_exp2(mp[s] - m);
        const float4 v = *reinterpret_cast<const float4 *>(mo + (s * kFuRows + row) * kFuRowStride + lane * 4);
        acc.x += v.x * w;
        acc.y += v.y * w;
        acc.z += v.z * w;
        acc.w += v.w * w;
        l += lp[s] * w;
    }
    m_out = m;
    l_out = l;
    return acc;
}

__global__ void __launch_bounds__(kDecWarps * 32, 1) decode_fused_kernel(DecArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_neff[kDecFusedMaxBatch];
    __shared__ int s_split[kDecFusedMaxBatch];
    __shared__ int s_shift[kDecFusedMaxBatch];
    __shared__ int s_tiles[kDecFusedMaxBatch];
    __shared__ int s_newrow[kDecFusedMaxBatch];
    __shared__ int s_n[kDecFusedMaxBatch];
    __shared__ int s_mode[kDecFusedMaxBatch];
    __shared__ const unsigned char *s_k[kDecFusedMaxBatch];
    __shared__ const unsigned char *s_v[kDecFusedMaxBatch];
    __shared__ unsigned s_ticket;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    float *mo = reinterpret_cast<float *>(smem + kFuStageBytes);
    float *mml = reinterpret_cast<float *>(smem + kFuStageBytes + kFuMergeOBytes);

    // Dependents are released at once: they get as far as their own wait (or their own prefetch).
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    // Everything the previous launch in the stream wrote is visible after the wait.
    if (!a.overlap) asm volatile("griddepcontrol.wait;\n" ::: "memory");
    const bool appending = a.k_new != nullptr;

    // ---- schedule -------------------------------------------------------------------------------
    if (tid < a.B) {
        const int b = tid;
        const ReqInfo r = req_info(a.ctx_len[b], a.mask[b * a.L + a.layer], a.S, a.W, a.layout, a.max_context,
                                   a.status);
        s_neff[b] = r.n_eff;
        s_split[b] = r.split;
        s_shift[b] = r.shift;
        s_tiles[b] = (r.n_eff + kFuCtaTok - 1) / kFuCtaTok;
        s_newrow[b] = dec_new_row(r, true, a.S, a.W, a.layout);   // cache row of position n - 1
        s_k[b] = (const unsigned char *)a.k_caches[b];
        s_v[b] = (const unsigned char *)a.v_caches[b];
        s_n[b] = r.n;
        s_mode[b] = r.mode;
    }
    __syncthreads();
    int total = 0;
    for (int b = 0; b < a.B; ++b) total += s_tiles[b] * a.Hkv;
    const int span = total > 0 ? (total + gridDim.x - 1) / gridDim.x : 1;
    const int u_begin = blockIdx.x * span;
    const int u_end = min(total, u_begin + span);
    const int n_units = max(u_end - u_begin, 0);

    // ---- iterators ------------------------------------------------------------------------------
    FuIt first = {0, 0, 0, 0, 1, 0};
    if (n_units > 0) {
        int b = 0, base = 0;
        while (u_begin >= base + s_tiles[b] * a.Hkv) {   // ends: u_begin < total
            base += s_tiles[b] * a.Hkv;
            ++b;
        }
        first.u = u_begin;
        first.b = b;
        first.base = base;
        first.tiles = s_tiles[b];
        first.head = (u_begin - base) / first.tiles;
        first.x = (u_begin - base) - first.head * first.tiles;
    }
    auto advance = [&](FuIt &it) {
        ++it.u;
        if (it.u >= u_end) return;
        if (++it.x == it.tiles) {
            it.x = 0;
            if (++it.head == a.Hkv) {
                it.head = 0;
                it.base += it.tiles * a.Hkv;
                do { ++it.b; } while (s_tiles[it.b] == 0);
                it.tiles = s_tiles[it.b];
            }
        }
    };

    unsigned char *my_smem = smem + (size_t)warp * kDecStages * kDecStageBytes;
    const uint32_t my_smem_u32 = smem_u32(my_smem);

    // loader: warp w brings tokens [x * 128 + 16 w, + 16) of (request, KV head), K and V.  The newest
    // row comes from k_new / v_new when this launch appends it; before the dependency wait (overlap mode)
    // it is left out and its place recorded in `patch`.
    FuIt lit = first;
    const int lc = lane & 15, lr0 = lane >> 4;
    uint32_t patch = 0;
    auto issue = [&](int stage, const bool before_wait) {
        const int b = lit.b, head = lit.head;
        const int n_eff = s_neff[b], split = s_split[b], shift = s_shift[b], newrow = s_newrow[b];
        const unsigned char *l_k = s_k[b] + (size_t)head * kRowBytes + lc * 16;
        const unsigned char *l_v = s_v[b] + (size_t)head * kRowBytes + lc * 16;
        const size_t row_bytes = (size_t)a.Hkv * kRowBytes;
        const int v0 = lit.x * kFuCtaTok + warp * kDecTile;
        const uint32_t sbase = my_smem_u32 + stage * kDecStageBytes;
#pragma unroll
        for (int i = 0; i < kDecTile / 2; ++i) {
            const int r = lr0 + 2 * i;
            const int v = v0 + r;
            const bool valid = v < n_eff;
            const int pos = valid ? (v >= split ? v + shift : v) : 0;
            const uint32_t dst = sbase + r * kRowBytes + ((lc ^ (r & 7)) << 4);
            if (a.touch != nullptr && valid && lc == 0 && head == 0)
                atomicOr(a.touch + (size_t)b * a.touch_words + (pos >> 5), 1u << (pos & 31));
            if (valid && pos == newrow && (before_wait || appending)) {
                if (before_wait) {
                    patch |= 1u << (stage * (kDecTile / 2) + i);
                } else {   // the token being appended by this launch
                    const size_t noff = ((size_t)b * a.Hkv + head) * kRowBytes + lc * 16;
                    cp_async16(dst, a.k_new + noff, 16);
                    cp_async16(dst + kDecTile * kRowBytes, a.v_new + noff, 16);
                }
            } else {
                cp_async16(dst, l_k + (size_t)pos * row_bytes, valid ? 16 : 0);
                cp_async16(dst + kDecTile * kRowBytes, l_v + (size_t)pos * row_bytes, valid ? 16 : 0);
            }
        }
        cp_async_commit();
    };

#pragma unroll
    for (int s = 0; s < kDecStages; ++s) {
        if (s < n_units) {
            issue(s, a.overlap != 0);
            advance(lit);
        } else {
            cp_async_commit();
        }
    }

    if (a.overlap) asm volatile("griddepcontrol.wait;\n" ::: "memory");

    // ---- after the wait: everything this launch writes, and the inputs the previous launch may have produced ----
    if (blockIdx.x == 0 && tid < a.B) {
        ReqInfo r;
        r.n = s_n[tid]; r.mode = s_mode[tid]; r.n_eff = s_neff[tid]; r.split = s_split[tid]; r.shift = s_shift[tid];
        dec_write_record(a.debug + tid * 8, r, a.layer, tid);
    }
    // inactive requests get a zero output row
    for (int b = blockIdx.x; b < a.B; b += gridDim.x) {
        if (s_tiles[b] != 0) continue;
        uint4 *dst = reinterpret_cast<uint4 *>(a.out + (size_t)b * a.Hq * kHeadDim);
        for (int i = tid; i < a.Hq * (kRowBytes / 16); i += blockDim.x) dst[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    // fused append: CTA b stores request b's newest K, V rows into the caches.  Nothing in this
    // launch reads those cache rows (the loaders take them from k_new / v_new).
    if (appending) {
        const int row_u4 = a.Hkv * (kRowBytes / 16);
        for (int b = blockIdx.x; b < a.B; b += gridDim.x) {
            const int nr = s_newrow[b];
            if (nr < 0) continue;
            uint4 *kd = (uint4 *)const_cast<unsigned char *>(s_k[b]) + (size_t)nr * row_u4;
            uint4 *vd = (uint4 *)const_cast<unsigned char *>(s_v[b]) + (size_t)nr * row_u4;
            const uint4 *ks = (const uint4 *)a.k_new + (size_t)b * row_u4;
            const uint4 *vs = (const uint4 *)a.v_new + (size_t)b * row_u4;
            for (int i = tid; i < row_u4; i += blockDim.x) {
                kd[i] = ks[i];
                vd[i] = vs[i];
            }
        }
    }
    if (n_units == 0) return;

    // consumer state
    FuIt cit = first;
    int cur_seg = -1, seg_b = 0, seg_head = 0, seg_us = 0, seg_ue = 0;
    float o[16][4];
    float m_r[2], l_r[2];
    uint32_t qf[8][4];
    const int g = lane >> 2, t4 = lane & 3;

    // Leaves a segment: CTA-level merge of the eight warps' states, one partial per query head to
    // global memory, a ticket; the last CTA of the segment merges all partials and writes the output.
    // Every warp of the CTA calls this at the same unit (the iterators do not depend on the warp).
    // `idle`: no tile loads are in flight any more (the CTA's last segment), so the stage memory can
    // take the partials.
    auto flush = [&](const bool idle) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            l_r[i] += __shfl_xor_sync(0xffffffffu, l_r[i], 1);
            l_r[i] += __shfl_xor_sync(0xffffffffu, l_r[i], 2);
        }
        const int c_first = seg_us / span, c_last = (seg_ue - 1) / span;
        const int n_part = c_last - c_first + 1;
        const size_t my_slot = (size_t)blockIdx.x + cur_seg;
        const int passes = a.G > kFuRows ? 2 : 1;
        for (int pass = 0; pass < passes; ++pass) {
            const int rows = min(a.G - pass * kFuRows, kFuRows);
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                if (i != pass) continue;
                float *po = mo + (warp * kFuRows + g) * kFuRowStride;
#pragma unroll
                for (int nt = 0; nt < 16; ++nt)
                    *reinterpret_cast<float2 *>(po + nt * 8 + 2 * t4) = make_float2(o[nt][2 * i], o[nt][2 * i + 1]);
                if (t4 == 0)
                    *reinterpret_cast<float2 *>(mml + (warp * kFuRows + g) * 2) = make_float2(m_r[i], l_r[i]);
            }
            __syncthreads();
            if (warp < rows) {
                float m, l;
                const float4 acc = fu_merge_row(mo, mml, warp, lane, m, l);
                const size_t e = my_slot * a.G + pass * kFuRows + warp;
                *reinterpret_cast<float4 *>(a.part_o + e * kHeadDim + lane * 4) = acc;
                if (lane == 0) *reinterpret_cast<float2 *>(a.part_ml + e * 2) = make_float2(m, l);
            }
            if (pass + 1 < passes) __syncthreads();   // the buffer is reused; after the last pass the ticket barrier does it
        }
        // One release-acquire ticket per CTA: the CTA's partial stores (ordered before thread 0 by the barrier)
        // become visible before the ticket is, and whoever draws the last ticket sees every partial.
        __syncthreads();
        if (tid == 0) {
            unsigned ticket;
            asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;\n" : "=r"(ticket) : "l"(a.tickets + cur_seg) : "memory");
            s_ticket = ticket;
        }
        __syncthreads();
        if (s_ticket != (unsigned)(n_part - 1)) return;
        // ---- last CTA of the segment ----------------------------------------------------------------
        // The segment's partials are one contiguous block: n_part * G rows from entry (c_first + cur_seg) * G.
        const size_t e_base = ((size_t)c_first + cur_seg) * a.G;
        const int n_rows = n_part * a.G;
        float2 *s_ml = reinterpret_cast<float2 *>(mml);
        const float *so = reinterpret_cast<const float *>(smem);
        if (idle && n_rows <= kFuStagedRows) {
            // No tile loads are in flight (the CTA's last segment): the block comes into the stage memory by one
            // round of asynchronous copies; then one warp per query head: weights 2^(m_p - m) first (lanes over
            // the partials), then the weighted sum with four partials in flight.  The loops stay rolled: this
            // code runs once per launch, and its size costs more than its arithmetic.
            float2 *st_ml = reinterpret_cast<float2 *>(smem + (size_t)kFuStagedRows * kHeadDim * 4);
            const unsigned char *src = reinterpret_cast<const unsigned char *>(a.part_o + e_base * kHeadDim);
            const uint32_t dst = smem_u32(smem);
            for (int c = tid; c < n_rows * (kHeadDim * 4 / 16); c += blockDim.x) cp_async16(dst + c * 16, src + (size_t)c * 16, 16);
            cp_async_commit();
            for (int i = tid; i < n_rows; i += blockDim.x) st_ml[i] = __ldcg(reinterpret_cast<const float2 *>(a.part_ml + (e_base + i) * 2));
            cp_async_wait<0>();
            __syncthreads();
            for (int r = warp; r < a.G; r += kDecWarps) {
                float m = kNegBig;
                for (int p = lane; p < n_part; p += 32) m = fmaxf(m, st_ml[p * a.G + r].x);
#pragma unroll
                for (int d = 16; d >= 1; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
                float l = 0.f;
                for (int p = lane; p < n_part; p += 32) {
                    const float2 ml = st_ml[p * a.G + r];
                    const float w = fast_exp2(ml.x - m);
                    st_ml[p * a.G + r].x = w;
                    l += ml.y * w;
                }
#pragma unroll
                for (int d = 16; d >= 1; d >>= 1) l += __shfl_xor_sync(0xffffffffu, l, d);
                __syncwarp();
                float4 acc[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                const float *row0 = so + (size_t)r * kHeadDim + lane * 4;
                const float2 *w0 = st_ml + r;
                int p = 0;
#pragma unroll 1
                for (; p + 4 <= n_part; p += 4) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float w = w0[(p + u) * a.G].x;
                        const float4 v = *reinterpret_cast<const float4 *>(row0 + (size_t)(p + u) * a.G * kHeadDim);
                        acc[u].x += v.x * w;
                        acc[u].y += v.y * w;
                        acc[u].z += v.z * w;
                        acc[u].w += v.w * w;
                    }
                }
#pragma unroll 1
                for (; p < n_part; ++p) {
                    const float w = w0[p * a.G].x;
                    const float4 v = *reinterpret_cast<const float4 *>(row0 + (size_t)p * a.G * kHeadDim);
                    acc[0].x += v.x * w;
                    acc[0].y += v.y * w;
                    acc[0].z += v.z * w;
                    acc[0].w += v.w * w;
                }
                const float inv = l > 0.f ? 1.0f / l : 0.f;
                uint2 pk;
                pk.x = pack_bf16((acc[0].x + acc[1].x + acc[2].x + acc[3].x) * inv, (acc[0].y + acc[1].y + acc[2].y + acc[3].y) * inv);
                pk.y = pack_bf16((acc[0].z + acc[1].z + acc[2].z + acc[3].z) * inv, (acc[0].w + acc[1].w + acc[2].w + acc[3].w) * inv);
                *reinterpret_cast<uint2 *>(a.out + ((size_t)seg_b * a.Hq + (size_t)seg_head * a.G + r) * kHeadDim + lane * 4) = pk;
            }
        } else {
            // Tile loads of the next segment are in flight (or the block is too large for the stage memory): warp w
            // folds partials w, w + 8, ... for every query head straight from global memory, then the eight warps'
            // results are merged like the per-CTA states above.
            for (int pass = 0; pass < passes; ++pass) {
                const int rows = min(a.G - pass * kFuRows, kFuRows);
                float4 acc[kFuRows];
                float mm[kFuRows], ll[kFuRows];
#pragma unroll
                for (int r = 0; r < kFuRows; ++r) {
                    acc[r] = make_float4(0.f, 0.f, 0.f, 0.f);
                    mm[r] = kNegBig;
                    ll[r] = 0.f;
                }
#pragma unroll 1
                for (int p = warp; p < n_part; p += kDecWarps) {
                    const size_t e0 = e_base + (size_t)p * a.G + pass * kFuRows;
                    float2 ml[kFuRows];
                    float4 v[kFuRows];
#pragma unroll
                    for (int r = 0; r < kFuRows; ++r) {
                        if (r < rows) {
                            ml[r] = __ldcg(reinterpret_cast<const float2 *>(a.part_ml + (e0 + r) * 2));
                            v[r] = __ldcg(reinterpret_cast<const float4 *>(a.part_o + (e0 + r) * kHeadDim + lane * 4));
                        } else {
                            ml[r] = make_float2(kNegBig, 0.f);
                            v[r] = make_float4(0.f, 0.f, 0.f, 0.f);
                        }
                    }
#pragma unroll
                    for (int r = 0; r < kFuRows; ++r) {
                        const float m_new = fmaxf(mm[r], ml[r].x);
                        const float sc = fast_exp2(mm[r] - m_new), sp = fast_exp2(ml[r].x - m_new);
                        acc[r].x = acc[r].x * sc + v[r].x * sp;
                        acc[r].y = acc[r].y * sc + v[r].y * sp;
                        acc[r].z = acc[r].z * sc + v[r].z * sp;
                        acc[r].w = acc[r].w * sc + v[r].w * sp;
                        ll[r] = ll[r] * sc + ml[r].y * sp;
                        mm[r] = m_new;
                    }
                }
#pragma unroll
                for (int r = 0; r < kFuRows; ++r) {
                    *reinterpret_cast<float4 *>(mo + (warp * kFuRows + r) * kFuRowStride + lane * 4) = acc[r];
                    if (lane == 0) s_ml[warp * kFuRows + r] = make_float2(mm[r], ll[r]);
                }
                __syncthreads();
                if (warp < rows) {
                    float m, l;
                    const float4 s4 = fu_merge_row(mo, mml, warp, lane, m, l);
                    const float inv = l > 0.f ? 1.0f / l : 0.f;
                    uint2 pk;
                    pk.x = pack_bf16(s4.x * inv, s4.y * inv);
                    pk.y = pack_bf16(s4.z * inv, s4.w * inv);
                    *reinterpret_cast<uint2 *>(a.out + ((size_t)seg_b * a.Hq + (size_t)seg_head * a.G + pass * kFuRows + warp) * kHeadDim +
                                               lane * 4) = pk;
                }
                __syncthreads();
            }
        }
        if (tid == 0) a.tickets[cur_seg] = 0u;   // ready for the next launch (stream order)
    };

    // Query rows of a segment: 16 rows of 256 bytes (rows >= G zero-filled) into this warp's part of the merge
    // buffer by asynchronous copies, swizzled like the K tiles, then A fragments by ldmatrix.
    const uint32_t q_smem = smem_u32(mo) + warp * (kFuRows * kFuRowStride * (int)sizeof(float));
    auto enter_segment = [&](const FuIt &it) {
        cur_seg = it.b * a.Hkv + it.head;
        seg_b = it.b;
        seg_head = it.head;
        seg_us = it.base + it.head * it.tiles;
        seg_ue = seg_us + it.tiles;
        dec_state_reset(o, m_r, l_r);
        const unsigned char *qb = reinterpret_cast<const unsigned char *>(a.q + ((size_t)it.b * a.Hq + (size_t)it.head * a.G) * kHeadDim);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = lr0 + 2 * i;
            const bool valid = r < a.G;
            cp_async16(q_smem + r * kRowBytes + ((lc ^ (r & 7)) << 4), qb + (valid ? (size_t)r * kRowBytes + lc * 16 : 0), valid ? 16 : 0);
        }
        cp_async_commit();
    };
    auto q_fragments = [&]() {   // after the copies of enter_segment have landed
        const int mi = lane >> 3, rr = lane & 7;
        const int row = rr + 8 * (mi & 1);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            const int chunk = 2 * kk + (mi >> 1);
            ldmatrix_x4(qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3], q_smem + row * kRowBytes + ((chunk ^ rr) << 4));
        }
    };
    enter_segment(cit);
    // the newest row of the tiles that were requested before the wait
    if (patch != 0) {
        FuIt pit = first;
        for (int st = 0; st < kDecStages && st < n_units; ++st) {
            const int b = pit.b, head = pit.head;
            const int v0 = pit.x * kFuCtaTok + warp * kDecTile;
#pragma unroll
            for (int i = 0; i < kDecTile / 2; ++i) {
                if (!((patch >> (st * (kDecTile / 2) + i)) & 1u)) continue;
                const int r = lr0 + 2 * i;
                const int v = v0 + r;
                const int pos = v >= s_split[b] ? v + s_shift[b] : v;
                const unsigned char *ksrc, *vsrc;
                if (appending) {
                    const size_t noff = ((size_t)b * a.Hkv + head) * kRowBytes + lc * 16;
                    ksrc = a.k_new + noff;
                    vsrc = a.v_new + noff;
                } else {
                    const size_t off = ((size_t)pos * a.Hkv + head) * kRowBytes + lc * 16;
                    ksrc = s_k[b] + off;
                    vsrc = s_v[b] + off;
                }
                unsigned char *dst = my_smem + st * kDecStageBytes + r * kRowBytes + ((lc ^ (r & 7)) << 4);
                *reinterpret_cast<uint4 *>(dst) = __ldcg(reinterpret_cast<const uint4 *>(ksrc));
                *reinterpret_cast<uint4 *>(dst + kDecTile * kRowBytes) = __ldcg(reinterpret_cast<const uint4 *>(vsrc));
            }
            advance(pit);
        }
    }
    cp_async_wait<0>();
    __syncwarp();
    q_fragments();

    // Three tiles are on their way before the first is used; tile t + 3 is requested into the slot of tile t
    // once that has been consumed.
    for (int t = 0; t < n_units; ++t) {
        cp_async_wait<kDecStages - 1>();
        __syncwarp();
        if (cit.b * a.Hkv + cit.head != cur_seg) {
            flush(false);
            enter_segment(cit);
            cp_async_wait<0>();
            __syncwarp();
            q_fragments();
        }
        const int n_valid = s_neff[cit.b] - (cit.x * kFuCtaTok + warp * kDecTile);   // <= 0: an empty trailing slice
        const uint32_t kb = my_smem_u32 + (t % kDecStages) * kDecStageBytes;
        dec_attend_tile(o, m_r, l_r, qf, kb, kb + kDecTile * kRowBytes, n_valid, a.scale_log2, lane);
        advance(cit);
        __syncwarp();
        if (t + kDecStages < n_units) {
            issue(t % kDecStages, false);
            advance(lit);
        } else {
            cp_async_commit();
        }
    }
    cp_async_wait<0>();
    __syncthreads();   // every warp is done with its stage memory
    flush(true);
}

}  // namespace

int decode_fused_setup(flux_plan *p)
{
    if (p->dev.smem_optin < kFuSmemBytes)
        return fail(FLUX_E_CUDA, "device offers %d bytes of shared memory per block, the single-launch decode needs %d",
                    p->dev.smem_optin, kFuSmemBytes);
    return check_cuda(cudaFuncSetAttribute(decode_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kFuSmemBytes),
                      "cudaFuncSetAttribute(decode_fused_kernel)");
}

int launch_decode_fused(flux_plan *p, const DecArgs &a, cudaStream_t st)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p->dec_ctas);
    cfg.blockDim = dim3(kDecWarps * 32);
    cfg.dynamicSmemBytes = kFuSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int rec = prof_begin(p, FLUX_KERNEL_DECODE, st);
    cudaError_t e = cudaLaunchKernelEx(&cfg, decode_fused_kernel, a);
    prof_end(p, rec, st);
    p->launches++;
    p->debug_records = a.B;
    return check_cuda(e, "single-launch decode kernel launch");
}

}  // namespace flux
