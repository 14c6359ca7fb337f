// Single-launch split-K decode (sm_100a), the default for batches of up to 32 requests.
//
// At batch 1 (the latency protocol of Appendix C.3) a sparse layer reads a few megabytes: the
// launch is bound by fixed costs, not by bandwidth, and a second launch that merges the split-K
// partials costs as much as the attention itself; on the batched workloads the second launch and its
// partial traffic still cost several per cent.  This kernel does the whole layer in one launch:
//
//  * work is split by (request, KV head, 128-token tile): a CTA streams one KV head's 256-byte
//    row pieces, its eight warps taking 16 tokens each, so a CTA produces partials for the G query
//    heads of one KV head only (a quarter or an eighth of what a whole-row CTA would write);
//  * when a CTA leaves a (request, KV head) segment its eight warps merge their flash-attention
//    states through shared memory into one partial (O, m, l) per query head;
//  * the CTA then announces itself on the segment's arrival counter and goes on; a CTA that covers a
//    whole segment alone writes the output rows straight away instead;
//  * when a CTA has finished all its tiles it takes its share of the merging: the i-th CTA of a
//    segment merges query head i (and i + the number of the segment's CTAs, ...) of that segment: it
//    waits -- a bounded spin on the arrival counter, which only CTAs of this same launch advance, none
//    of which waits for anything before announcing itself -- until all the segment's CTAs have announced
//    themselves, copies the head's partials into its idle stage memory and merges them (Eq. 1 / Eq. 2 are
//    sums over disjoint key sets, which merge by rescaling with 2^(m_p - m)).  The merge of a segment is
//    thus spread over as many SMs as it has query heads, each reading a seventh (G = 7) of the partials.
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
// the kernel's static shared memory (per-request tables for kDecFusedMaxBatch requests) takes the rest of the 227 KB
static_assert(kFuSmemBytes + 48 * kDecFusedMaxBatch <= 232448, "shared memory per CTA");
// partial rows (512 bytes of O and 8 bytes of (m, l) each) the idle stage memory takes for the last CTA's merge
constexpr int kFuStagedRows = kFuStageBytes / (kHeadDim * 4 + 8);
constexpr long long kFuWaitCycles = 2000000000ll;   // bound of the wait for a segment's arrivals (about a second)
constexpr int kFuMaxDuties = 2;                      // segments a CTA shares with other CTAs: the first and the last of its span

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
    __shared__ int s_duty[kFuMaxDuties][5];   // segment, first CTA, CTAs, request, KV head of the segments to help merge
    __shared__ int s_n_duty;
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        s_n_duty = 0;
        s_abort = 0;
    }
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
    // Merges query heads r_first, r_first + r_step, ... of a segment whose partials come from n_part CTAs (c_first ...):
    // waits until all of them have announced themselves, brings a head's partials into the stage memory (idle by then),
    // folds them, writes the output row.  `helpers` CTAs do this for the segment; the last of them to get here puts
    // the counters back to zero.  False when the wait ran out.
    auto help = [&](int seg, int c_first, int n_part, int db, int dh, int r_first, int r_step, int helpers) -> bool {
        // Wait until every CTA of the segment has announced itself (they all do, unconditionally, when they leave the
        // segment).  The order in which the helpers get here decides who puts the counters back to zero: the last one,
        // which knows that nobody will look at them again.
        unsigned order = 0;
        if (tid == 0) {
            const long long t0 = clock64();
            unsigned seen;
            do {
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(seen) : "l"(a.tickets + seg) : "memory");
                if (seen < (unsigned)n_part && clock64() - t0 > kFuWaitCycles) {
                    atomicOr(a.status, FLUX_STATUS_WAIT_EXPIRED);
                    s_abort = 1;
                    break;
                }
            } while (seen < (unsigned)n_part);
            // (the answer is needed only at the very end: nothing waits for this round trip)
            asm volatile("atom.relaxed.gpu.global.add.u32 %0, [%1], 1;\n" : "=r"(order) : "l"(a.done + seg) : "memory");
        }
        __syncthreads();
        if (s_abort) return false;
        const size_t e_base = ((size_t)c_first + seg) * a.G;      // partial p of query head r: entry e_base + p * G + r
        float *st_o = reinterpret_cast<float *>(smem);
        float2 *st_ml = reinterpret_cast<float2 *>(smem + (size_t)kFuStagedRows * kHeadDim * 4);
        for (int r = r_first; r < a.G; r += r_step) {
            for (int p0 = 0; p0 < n_part; p0 += kFuStagedRows) {     // (one round unless a head has hundreds of partials)
                const int np = min(n_part - p0, kFuStagedRows);
                for (int c = tid; c < np * 32; c += blockDim.x) {
                    const int p = c >> 5, piece = c & 31;
                    cp_async16(smem_u32(st_o) + (uint32_t)c * 16u, a.part_o + (e_base + (size_t)(p0 + p) * a.G + r) * kHeadDim + piece * 4, 16);
                }
                cp_async_commit();
                for (int p = tid; p < np; p += blockDim.x)
                    st_ml[p] = __ldcg(reinterpret_cast<const float2 *>(a.part_ml + (e_base + (size_t)(p0 + p) * a.G + r) * 2));
                cp_async_wait<0>();
                __syncthreads();
                // warp w folds partials w, w + 8, ... ; the warps' results go through the merge buffers; a later round
                // of the same head starts from the merged state of the rounds before (kept by warp 0)
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                float m = kNegBig, l = 0.f;
                if (p0 > 0 && warp == 0) {
                    acc = *reinterpret_cast<const float4 *>(mo + (size_t)kDecWarps * kFuRows * kFuRowStride - kHeadDim + lane * 4);
                    m = mml[kDecWarps * kFuRows * 2 - 2];
                    l = mml[kDecWarps * kFuRows * 2 - 1];
                }
#pragma unroll 2
                for (int p = warp; p < np; p += kDecWarps) {
                    const float2 ml = st_ml[p];
                    const float4 v = *reinterpret_cast<const float4 *>(st_o + (size_t)p * kHeadDim + lane * 4);
                    const float m_new = fmaxf(m, ml.x);
                    const float sc = fast_exp2(m - m_new), sp = fast_exp2(ml.x - m_new);
                    acc.x = acc.x * sc + v.x * sp;
                    acc.y = acc.y * sc + v.y * sp;
                    acc.z = acc.z * sc + v.z * sp;
                    acc.w = acc.w * sc + v.w * sp;
                    l = l * sc + ml.y * sp;
                    m = m_new;
                }
                *reinterpret_cast<float4 *>(mo + (warp * kFuRows) * kFuRowStride + lane * 4) = acc;
                if (lane == 0) *reinterpret_cast<float2 *>(mml + (warp * kFuRows) * 2) = make_float2(m, l);
                __syncthreads();
                if (warp == 0) {
                    float mm, ll;
                    const float4 s4 = fu_merge_row(mo, mml, 0, lane, mm, ll);
                    if (p0 + np < n_part) {          // more rounds to come: keep the state at the end of the buffers
                        *reinterpret_cast<float4 *>(mo + (size_t)kDecWarps * kFuRows * kFuRowStride - kHeadDim + lane * 4) = s4;
                        if (lane == 0) {
                            mml[kDecWarps * kFuRows * 2 - 2] = mm;
                            mml[kDecWarps * kFuRows * 2 - 1] = ll;
                        }
                    } else {
                        const float inv = ll > 0.f ? 1.0f / ll : 0.f;
                        uint2 pk;
                        pk.x = pack_bf16(s4.x * inv, s4.y * inv);
                        pk.y = pack_bf16(s4.z * inv, s4.w * inv);
                        *reinterpret_cast<uint2 *>(a.out + ((size_t)db * a.Hq + (size_t)dh * a.G + r) * kHeadDim + lane * 4) = pk;
                    }
                }
                __syncthreads();
            }
        }
        if (tid == 0 && order == (unsigned)(helpers - 1)) {   // ready for the next launch (stream order)
            a.tickets[seg] = 0u;
            a.done[seg] = 0u;
        }
        return true;
    };

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
    auto flush = [&]() {
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
                if (n_part == 1) {   // this CTA has the whole segment: the output row itself
                    const float inv = l > 0.f ? 1.0f / l : 0.f;
                    uint2 pk;
                    pk.x = pack_bf16(acc.x * inv, acc.y * inv);
                    pk.y = pack_bf16(acc.z * inv, acc.w * inv);
                    *reinterpret_cast<uint2 *>(a.out + ((size_t)seg_b * a.Hq + (size_t)seg_head * a.G + pass * kFuRows + warp) * kHeadDim +
                                               lane * 4) = pk;
                } else {
                    const size_t e = my_slot * a.G + pass * kFuRows + warp;
                    *reinterpret_cast<float4 *>(a.part_o + e * kHeadDim + lane * 4) = acc;
                    if (lane == 0) *reinterpret_cast<float2 *>(a.part_ml + e * 2) = make_float2(m, l);
                }
            }
            if (pass + 1 < passes || n_part == 1) __syncthreads();   // the buffer is reused (else the barrier below does it)
        }
        if (n_part == 1) return;
        // the CTA's partial stores (ordered before thread 0 by the barrier) become visible before its arrival is
        __syncthreads();
        if (tid == 0) {
            asm volatile("red.release.gpu.global.add.u32 [%0], 1;\n" ::"l"(a.tickets + cur_seg) : "memory");
            const int d = s_n_duty;       // at most two segments of a span are shared with other CTAs
            s_duty[d][0] = cur_seg; s_duty[d][1] = c_first; s_duty[d][2] = n_part; s_duty[d][3] = seg_b; s_duty[d][4] = seg_head;
            s_n_duty = d + 1;
        }
        __syncthreads();
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
            flush();
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
    flush();
    __syncthreads();   // every warp is done with its stage memory and the merge buffers

    // ---- this CTA's share of the merging ---------------------------------------------------------------
    const int n_duty = s_n_duty;
    for (int d = 0; d < n_duty; ++d) {
        const int c_first = s_duty[d][1], n_part = s_duty[d][2];
        const int idx = (int)blockIdx.x - c_first;       // this CTA's place among the segment's CTAs
        if (idx >= a.G) continue;                        // more CTAs than query heads: the later ones have nothing to merge
        if (!help(s_duty[d][0], c_first, n_part, s_duty[d][3], s_duty[d][4], idx, n_part, n_part < a.G ? n_part : a.G)) return;
    }
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
