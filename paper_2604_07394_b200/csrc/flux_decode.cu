// Split-K flash-decode for a batch with mixed FA / SA layers (sm_100a).
//
// One launch serves every request of the batch for one layer.  A request in FA
// mode streams its whole KV cache (Eq. 1); a request in SA mode streams only the
// sink rows and the window rows (Eq. 2 with the streaming subset; Appendix C.3:
// a sparse layer reads only the rows it keeps).  The kept rows of
// all requests are laid end to end in units of `slices * kDecTile` tokens and cut
// into gridDim.x equal spans, so every SM streams the same number of bytes
// whatever the mix of modes and lengths.  Inside a CTA each warp owns one KV
// head (and one token slice), so the CTA as a whole reads whole token rows of the
// token-major cache: contiguous, 16-byte vectorised cp.async traffic, no
// block-level barrier anywhere.  Each warp keeps a flash-attention state
// (running max, sum, fp32 accumulator) for the G query heads of its KV head,
// computes QK^T and PV with bf16 tensor-core MMAs (m16n8k16, rows padded to 16),
// and writes one partial (O, m, l) per segment it touched; a small combine kernel
// merges the partials (the split-K identity: sums over disjoint key sets merge by
// rescaling with exp(m_p - m)).
#include <math.h>

#include <mutex>

#include "flux_decode_common.h"

namespace flux {

int launch_decode_fused(flux_plan *p, const DecArgs &a, cudaStream_t st);   // flux_decode_fused.cu

namespace {

// position of the unit a warp is loading or consuming
struct UnitIt {
    int u;      // global unit index
    int b;      // request
    int hg;     // head group
    int x;      // CTA tile inside the request
    int tiles;  // CTA tiles of request b
};

__global__ void __launch_bounds__(kDecWarps * 32, 1) decode_kernel(DecArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_prefix[kMaxBatch + 1];
    __shared__ int s_neff[kMaxBatch];
    __shared__ int s_split[kMaxBatch];
    __shared__ int s_shift[kMaxBatch];
    __shared__ int s_units[kMaxBatch];
    __shared__ int s_newrow[kMaxBatch];   // fused append: cache row of the newest token (-1: none)

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int hpc = a.Hkv < kDecWarps ? a.Hkv : kDecWarps;
    const int slices = kDecWarps / hpc;
    const int n_hg = (a.Hkv + hpc - 1) / hpc;
    const int cta_tok = slices * kDecTile;

    // ---- schedule: units per request, prefix sum, equal spans -------------------------------
    for (int b = tid; b < a.B; b += blockDim.x) {
        int mode_raw;
        if (a.head_mask != nullptr) {   // the request is walked over its full length if any head is dense
            mode_raw = 0;
            for (int h = 0; h < a.Hkv; ++h) {
                const int mh = a.head_mask[b * a.Hkv + h];
                if (mh > 1) atomicOr(a.status, FLUX_STATUS_BAD_MASK);
                mode_raw |= (mh != 0);
            }
        } else {
            mode_raw = a.mask[b * a.L + a.layer];
        }
        ReqInfo r = req_info(a.ctx_len[b], mode_raw, a.S, a.W, a.layout, a.max_context, a.status);
        if (a.key_begin != nullptr) dec_restrict(r, a.key_begin[b], a.key_end[b], a.S, a.W);
        s_neff[b] = r.n_eff;
        s_split[b] = r.split;
        s_shift[b] = r.shift;
        s_units[b] = (r.n_eff + cta_tok - 1) / cta_tok * n_hg;
        s_newrow[b] = dec_new_row(r, a.k_new != nullptr, a.S, a.W, a.layout);
        if (blockIdx.x == 0) dec_write_record(a.debug + b * 8, r, a.layer, b);
    }
    __syncthreads();
    if (warp == 0) {
        const int chunk = (a.B + 31) / 32;
        const int lo = lane * chunk, hi = min(a.B, lo + chunk);
        int sum = 0;
        for (int b = lo; b < hi; ++b) sum += s_units[b];
        int incl = sum;
        for (int d = 1; d < 32; d <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += t;
        }
        int run = incl - sum;
        for (int b = lo; b < hi; ++b) {
            s_prefix[b] = run;
            run += s_units[b];
        }
        if (lane == 31) s_prefix[a.B] = incl;
    }
    __syncthreads();
    const int total = s_prefix[a.B];
    const int span = total > 0 ? (total + gridDim.x - 1) / gridDim.x : 1;
    if (blockIdx.x == 0) {
        for (int b = tid; b <= a.B; b += blockDim.x) a.sched[b] = s_prefix[b];
        if (tid == 0) a.sched[a.B + 1] = span;
    }
    // fused append: CTA b stores request b's newest K, V rows into the caches.  Nothing in this
    // launch reads those cache rows (the loaders below take them from k_new / v_new).
    if (a.k_new != nullptr) {
        const int row_u4 = a.Hkv * (kRowBytes / 16);
        for (int b = blockIdx.x; b < a.B; b += gridDim.x) {
            const int nr = s_newrow[b];
            if (nr < 0) continue;
            uint4 *kd = (uint4 *)const_cast<void *>(a.k_caches[b]) + (size_t)nr * row_u4;
            uint4 *vd = (uint4 *)const_cast<void *>(a.v_caches[b]) + (size_t)nr * row_u4;
            const uint4 *ks = (const uint4 *)a.k_new + (size_t)b * row_u4;
            const uint4 *vs = (const uint4 *)a.v_new + (size_t)b * row_u4;
            for (int i = tid; i < row_u4; i += blockDim.x) {
                kd[i] = ks[i];
                vd[i] = vs[i];
            }
        }
    }
    const int u_begin = blockIdx.x * span;
    const int u_end = min(total, u_begin + span);
    if (u_begin >= u_end) return;
    const int slice = warp / hpc, hw = warp % hpc;
    if (slice >= slices) return;

    // ---- iterators ------------------------------------------------------------------------------
    UnitIt first;
    {
        int lo = 0, hi = a.B - 1;  // last b with prefix[b] <= u_begin and units > 0
        while (lo < hi) {
            int mid = (lo + hi + 1) >> 1;
            if (s_prefix[mid] <= u_begin) lo = mid; else hi = mid - 1;
        }
        while (s_units[lo] == 0 && lo + 1 < a.B) ++lo;  // cannot trigger: u_begin < total
        first.u = u_begin;
        first.b = lo;
        first.tiles = s_units[lo] / n_hg;
        const int off = u_begin - s_prefix[lo];
        first.hg = off / first.tiles;
        first.x = off % first.tiles;
    }
    auto advance = [&](UnitIt &it) {
        ++it.u;
        if (it.u >= u_end) return;
        if (++it.x == it.tiles) {
            it.x = 0;
            if (++it.hg == n_hg) {
                it.hg = 0;
                do { ++it.b; } while (s_units[it.b] == 0);
                it.tiles = s_units[it.b] / n_hg;
            }
        }
    };

    unsigned char *my_smem = smem + (size_t)warp * kDecStages * kDecStageBytes;
    const uint32_t my_smem_u32 = smem_u32(my_smem);

    // Rows a KV head reads of request b.  Routed calls: the request's values.  Head-level mode: a
    // sparse head inside a request that is walked densely keeps sink + window (full cache layout),
    // so its warps run out of rows after the first few tiles of the request and idle.
    auto head_rows = [&](int b, int head, int &n_eff, int &split, int &shift) {
        n_eff = s_neff[b];
        split = s_split[b];
        shift = s_shift[b];
        if (a.head_mask != nullptr && n_eff > a.S + a.W && a.head_mask[b * a.Hkv + head] == 0) {
            shift = n_eff - a.W - a.S;
            split = a.S;
            n_eff = a.S + a.W;
        }
    };

    // loader state
    UnitIt lit = first;
    int l_b = -1;
    const unsigned char *l_k = nullptr, *l_v = nullptr;
    const int lc = lane & 15, lr0 = lane >> 4;
    auto issue = [&](int stage) {
        const int head = lit.hg * hpc + hw;
        if (head < a.Hkv) {
            if (lit.b != l_b) {
                l_b = lit.b;
                l_k = (const unsigned char *)a.k_caches[l_b];
                l_v = (const unsigned char *)a.v_caches[l_b];
            }
            int n_eff, split, shift;
            head_rows(l_b, head, n_eff, split, shift);
            const int newrow = s_newrow[l_b];
            const int v0 = (lit.x * slices + slice) * kDecTile;
            const uint32_t sbase = my_smem_u32 + stage * kDecStageBytes;
#pragma unroll
            for (int i = 0; i < kDecTile / 2; ++i) {
                const int r = lr0 + 2 * i;
                const int v = v0 + r;
                const bool valid = v < n_eff;
                const int pos = valid ? (v >= split ? v + shift : v) : 0;
                const size_t off = ((size_t)pos * a.Hkv + head) * kRowBytes + lc * 16;
                const uint32_t dst = sbase + r * kRowBytes + ((lc ^ (r & 7)) << 4);
                if (a.touch != nullptr && valid && lc == 0 && head == 0)
                    atomicOr(a.touch + (size_t)l_b * a.touch_words + (pos >> 5), 1u << (pos & 31));
                if (valid && pos == newrow) {   // the token being appended by this launch
                    const size_t noff = ((size_t)l_b * a.Hkv + head) * kRowBytes + lc * 16;
                    cp_async16(dst, a.k_new + noff, 16);
                    cp_async16(dst + kDecTile * kRowBytes, a.v_new + noff, 16);
                } else {
                    cp_async16(dst, l_k + off, valid ? 16 : 0);
                    cp_async16(dst + kDecTile * kRowBytes, l_v + off, valid ? 16 : 0);
                }
            }
        }
        cp_async_commit();
    };

    const int n_units = u_end - u_begin;
#pragma unroll
    for (int s = 0; s < kDecStages - 1; ++s) {
        if (s < n_units) {
            issue(s);
            advance(lit);
        } else {
            cp_async_commit();
        }
    }

    // consumer state
    UnitIt cit = first;
    int cur_seg = -1;
    bool cur_active = false;
    float o[16][4];
    float m_r[2], l_r[2];
    uint32_t qf[8][4];
    const int g = lane >> 2, t4 = lane & 3;

    auto flush = [&]() {
        if (cur_seg < 0 || !cur_active) return;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            l_r[i] += __shfl_xor_sync(0xffffffffu, l_r[i], 1);
            l_r[i] += __shfl_xor_sync(0xffffffffu, l_r[i], 2);
        }
        const size_t slot = ((size_t)blockIdx.x + cur_seg) * kDecWarps + warp;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int row = g + 8 * i;
            if (row < a.G) {
                float *po = a.part_o + (slot * a.G + row) * kHeadDim;
#pragma unroll
                for (int nt = 0; nt < 16; ++nt)
                    *reinterpret_cast<float2 *>(po + nt * 8 + 2 * t4) =
                        make_float2(o[nt][2 * i], o[nt][2 * i + 1]);
                if (t4 == 0) {
                    float *pm = a.part_ml + (slot * a.G + row) * 2;
                    pm[0] = m_r[i];
                    pm[1] = l_r[i];
                }
            }
        }
    };

    for (int t = 0; t < n_units; ++t) {
        cp_async_wait<kDecStages - 2>();
        __syncwarp();
        if (t + kDecStages - 1 < n_units) {
            issue((t + kDecStages - 1) % kDecStages);
            advance(lit);
        } else {
            cp_async_commit();
        }

        const int seg = cit.b * n_hg + cit.hg;
        if (seg != cur_seg) {
            flush();
            cur_seg = seg;
            const int head = cit.hg * hpc + hw;
            cur_active = head < a.Hkv;
            if (cur_active) {
                dec_state_reset(o, m_r, l_r);
                dec_load_q(qf, a.q + ((size_t)cit.b * a.Hq + (size_t)head * a.G) * kHeadDim, a.G, lane);
            }
        }

        int n_valid = 0;
        if (cur_active) {
            int n_eff, split, shift;
            head_rows(cit.b, cit.hg * hpc + hw, n_eff, split, shift);
            n_valid = n_eff - (cit.x * slices + slice) * kDecTile;  // may be <= 0 for a trailing empty slice
        }
        // (head-level mode: a sparse head's warp has nothing to do on most tiles of a dense walk)
        if (cur_active && (a.head_mask == nullptr || n_valid > 0)) {
            const int stage = t % kDecStages;
            const uint32_t kb = my_smem_u32 + stage * kDecStageBytes;
            dec_attend_tile(o, m_r, l_r, qf, kb, kb + kDecTile * kRowBytes, n_valid, a.scale_log2, lane);
        }
        advance(cit);
    }
    flush();
    cp_async_wait<0>();
}

// Merge the partials of one (request, query head) and write the bf16 output row.
// Split-K combine: m = max m_p, l = sum l_p 2^(m_p - m), O = sum O_p 2^(m_p - m) / l over the
// partials of one (request, query head).  One CTA per (request, head); its 16 warps take the
// partials round-robin, eight at a time with all loads issued before any is used (at batch 1 one
// head has a few hundred partials, and a loop of dependent loads would cost more than the decode
// kernel itself), then the warps' results are merged through shared memory.
constexpr int kCombWarps = 16;

// Pushed pieces: channel d of the merged row of (request, head) `row` goes to slot push_rank of every gather buffer
// -- this GPU's own and its peers', plain stores over NVLink -- and thread 0 adds (m, l).
__device__ __forceinline__ void push_row(const DecArgs &a, size_t row, int d, float o, float m, float l)
{
    const size_t e = (size_t)a.push_rank * a.B * a.Hq + row;
    for (int p = 0; p < a.push_world; ++p) {
        a.push_o[p][e * kHeadDim + d] = o;
        if (d == 0) *reinterpret_cast<float2 *>(a.push_ml[p] + e * 2) = make_float2(m, l);
    }
}
// Called by every thread of every CTA of the merge launch once its stores are issued: the CTA that gets here last
// tells every gather buffer's owner that this rank's piece is complete (flag = push_seq, released at system scope
// after every CTA's stores, which each CTA fenced at system scope before it took its ticket).
__device__ __forceinline__ void push_signal(const DecArgs &a)
{
    __threadfence_system();
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned ticket;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;\n" : "=r"(ticket) : "l"(a.push_ticket) : "memory");
        if (ticket == gridDim.x - 1) {
            *a.push_ticket = 0u;
            for (int p = 0; p < a.push_world; ++p)
                asm volatile("st.release.sys.global.u32 [%0], %1;\n" ::"l"(a.push_flags[p] + a.push_rank), "r"(a.push_seq) : "memory");
        }
    }
}

__global__ void __launch_bounds__(kCombWarps * 32) decode_combine_kernel(DecArgs a)
{
    __shared__ float s_o[kCombWarps][kHeadDim];
    __shared__ float s_m[kCombWarps], s_l[kCombWarps];
    const int b = blockIdx.x / a.Hq, h = blockIdx.x % a.Hq;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hpc = a.Hkv < kDecWarps ? a.Hkv : kDecWarps;
    const int slices = kDecWarps / hpc;
    const int n_hg = (a.Hkv + hpc - 1) / hpc;
    __nv_bfloat16 *dst = a.out + ((size_t)b * a.Hq + h) * kHeadDim;

    const int ustart = a.sched[b], uend = a.sched[b + 1], span = a.sched[a.B + 1];
    const int units = uend - ustart;
    float *pdst_o = a.pout_o ? a.pout_o + ((size_t)b * a.Hq + h) * kHeadDim : nullptr;
    if (units == 0) {  // inactive request (or, in a partial call, no key of the range is kept): nothing to add
        if (a.push_world > 0) {
            if (threadIdx.x < kHeadDim) push_row(a, (size_t)b * a.Hq + h, threadIdx.x, 0.f, kNegBig, 0.f);
            push_signal(a);
            return;
        }
        if (threadIdx.x < kHeadDim) {
            if (pdst_o) pdst_o[threadIdx.x] = 0.f; else dst[threadIdx.x] = __float2bfloat16(0.f);
        }
        if (pdst_o && threadIdx.x == 0)
            *reinterpret_cast<float2 *>(a.pout_ml + ((size_t)b * a.Hq + h) * 2) = make_float2(kNegBig, 0.f);
        return;
    }
    const int tiles = units / n_hg;
    const int kvh = h / a.G, r = h % a.G;
    const int hg = kvh / hpc, hw = kvh % hpc;
    const int us = ustart + hg * tiles, ue = us + tiles;
    const int c_first = us / span, c_last = (ue - 1) / span;
    const int seg = b * n_hg + hg;
    const int n_part = (c_last - c_first + 1) * slices;

    float m = kNegBig, l = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    constexpr int kUnroll = 8;
    // Partial p of this head sits in the slot of CTA c_first + p / slices, slice p % slices.  slices is a
    // power of two that divides the warp count, so a warp always meets the same slice and walks the CTAs
    // with a constant stride: all addressing is 32-bit adds on a base computed once.
    const int sh = 31 - __clz(slices);
    const int step_c = kCombWarps >> sh;                                    // CTAs between two partials of a warp
    const int slot0 = (c_first + seg + (warp >> sh)) * kDecWarps + hw + hpc * (warp & (slices - 1));
    const float *po = a.part_o + ((size_t)slot0 * a.G + r) * kHeadDim + lane * 4;
    const float *pm = a.part_ml + ((size_t)slot0 * a.G + r) * 2;
    const int stride_o = step_c * kDecWarps * a.G * kHeadDim, stride_m = step_c * kDecWarps * a.G * 2;
    for (int p0 = warp; p0 < n_part; p0 += kCombWarps * kUnroll) {
        float mp[kUnroll], lp[kUnroll];
        float4 op[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (p0 + u * kCombWarps < n_part) {
                const float2 ml = *reinterpret_cast<const float2 *>(pm + u * stride_m);
                mp[u] = ml.x;
                lp[u] = ml.y;
                op[u] = *reinterpret_cast<const float4 *>(po + u * stride_o);
            } else {
                mp[u] = kNegBig;
                lp[u] = 0.f;
                op[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        po += kUnroll * stride_o;
        pm += kUnroll * stride_m;
        float m_new = m;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) m_new = fmaxf(m_new, mp[u]);
        const float so = fast_exp2(m - m_new);
        acc.x *= so; acc.y *= so; acc.z *= so; acc.w *= so;
        l *= so;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const float sp = fast_exp2(mp[u] - m_new);
            acc.x += op[u].x * sp;
            acc.y += op[u].y * sp;
            acc.z += op[u].z * sp;
            acc.w += op[u].w * sp;
            l += lp[u] * sp;
        }
        m = m_new;
    }
    *reinterpret_cast<float4 *>(&s_o[warp][lane * 4]) = acc;
    if (lane == 0) {
        s_m[warp] = m;
        s_l[warp] = l;
    }
    __syncthreads();
    if (threadIdx.x >= kHeadDim) {
        if (a.push_world > 0) push_signal(a);
        return;
    }
    const int d = threadIdx.x;
    float mm = kNegBig;
#pragma unroll
    for (int w = 0; w < kCombWarps; ++w) mm = fmaxf(mm, s_m[w]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < kCombWarps; ++w) {
        const float sc = fast_exp2(s_m[w] - mm);
        num += s_o[w][d] * sc;
        den += s_l[w] * sc;
    }
    if (a.push_world > 0) {   // pushed piece: the merged state goes straight into every rank's gather buffer
        push_row(a, (size_t)b * a.Hq + h, d, num, mm, den);
        push_signal(a);
    } else if (pdst_o) {   // partial call: the merged state itself (O unnormalised), for flux_attn_combine
        pdst_o[d] = num;
        if (d == 0) *reinterpret_cast<float2 *>(a.pout_ml + ((size_t)b * a.Hq + h) * 2) = make_float2(mm, den);
    } else {
        dst[d] = __float2bfloat16(den > 0.f ? num / den : 0.f);
    }
}

// Merges n_sets partial evaluations of the same (request, query head) rows -- each (O unnormalised, m, l) over a
// disjoint set of keys -- into the bf16 output: m = max m_s, O = sum O_s 2^(m_s - m), l likewise, out = O / l.
// Sets are laid out [set][row]; one warp per row, four channels per lane, the sets taken in order.
// With `flags` (flux_attn_combine_wait) the sets are pieces that other GPUs store into this buffer: set s is complete
// once flags[s] holds `seq` (its owner releases the flag at system scope after its stores), and every CTA first waits for
// all flags -- a bounded spin: the writers are kernels on other GPUs (or earlier launches on this one), which never wait
// for this kernel -- and gives up with FLUX_STATUS_WAIT_EXPIRED, writing nothing, when the limit runs out.
__global__ void __launch_bounds__(256) combine_sets_kernel(const float *po, const float *pml, int n_sets, int n_rows,
                                                           __nv_bfloat16 *__restrict__ out, const uint32_t *flags, uint32_t seq,
                                                           long long wait_cycles, uint32_t *status)
{
    if (flags != nullptr) {
        __shared__ int s_ok;
        if (threadIdx.x == 0) {
            int ok = 1;
            const long long t0 = clock64();
            for (int s = 0; s < n_sets && ok; ++s) {
                for (;;) {
                    uint32_t v;
                    asm volatile("ld.acquire.sys.global.u32 %0, [%1];\n" : "=r"(v) : "l"(flags + s) : "memory");
                    if (v == seq) break;
                    if (clock64() - t0 > wait_cycles) {
                        atomicOr(status, FLUX_STATUS_WAIT_EXPIRED);
                        ok = 0;
                        break;
                    }
                }
            }
            s_ok = ok;
        }
        __syncthreads();
        if (!s_ok) return;
    }
    const int row = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    if (row >= n_rows) return;
    float m = kNegBig;
    for (int s = 0; s < n_sets; ++s) m = fmaxf(m, pml[((size_t)s * n_rows + row) * 2]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
    for (int s = 0; s < n_sets; ++s) {
        const float2 ml = *reinterpret_cast<const float2 *>(pml + ((size_t)s * n_rows + row) * 2);
        const float w = fast_exp2(ml.x - m);
        const float4 v = *reinterpret_cast<const float4 *>(po + ((size_t)s * n_rows + row) * kHeadDim + lane * 4);
        acc.x += v.x * w;
        acc.y += v.y * w;
        acc.z += v.z * w;
        acc.w += v.w * w;
        l += ml.y * w;
    }
    const float inv = l > 0.f ? 1.0f / l : 0.f;
    uint2 pk;
    pk.x = pack_bf16(acc.x * inv, acc.y * inv);
    pk.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2 *>(out + (size_t)row * kHeadDim + lane * 4) = pk;
}

constexpr int kDecSmemBytes = kDecWarps * kDecStages * kDecStageBytes;

}  // namespace

int decode_setup(flux_plan *p)
{
    if (p->dev.smem_optin < kDecSmemBytes)
        return fail(FLUX_E_CUDA, "device offers %d bytes of shared memory per block, decode needs %d",
                    p->dev.smem_optin, kDecSmemBytes);
    return check_cuda(cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kDecSmemBytes),
                      "cudaFuncSetAttribute(decode_kernel)");
}

int launch_combine_sets(flux_plan *p, const float *po, const float *pml, int n_sets, int n_rows, void *out, cudaStream_t st,
                        const uint32_t *flags, uint32_t seq, long long wait_cycles)
{
    combine_sets_kernel<<<(n_rows + 7) / 8, 256, 0, st>>>(po, pml, n_sets, n_rows, (__nv_bfloat16 *)out, flags, seq, wait_cycles,
                                                         (uint32_t *)((char *)p->ws + p->lay.status));
    p->launches++;
    return check_cuda(cudaGetLastError(), "partial-set combine kernel launch");
}

int launch_decode(flux_plan *p, int layer, int B, const void *q, const void *const *k_caches,
                  const void *const *v_caches, const int32_t *ctx_len, void *out, cudaStream_t st,
                  const void *k_new, const void *v_new, const uint8_t *head_mask, const DecPartial *part)
{
    const flux_config &c = p->cfg;
    char *ws = (char *)p->ws;
    DecArgs a;
    a.q = (const __nv_bfloat16 *)q;
    a.k_caches = k_caches;
    a.v_caches = v_caches;
    a.ctx_len = ctx_len;
    a.mask = p->d_mask;
    a.B = B; a.L = c.n_layers; a.layer = layer; a.Hq = c.n_q_heads; a.Hkv = c.n_kv_heads;
    a.G = p->G; a.S = c.sink; a.W = c.window; a.layout = c.kv_layout; a.max_context = c.max_context;
    a.scale_log2 = p->scale_log2;
    a.part_o = (float *)(ws + p->lay.part_o);
    a.part_ml = (float *)(ws + p->lay.part_ml);
    a.debug = (int32_t *)(ws + p->lay.debug);
    a.sched = (int32_t *)(ws + p->lay.sched);
    a.status = (uint32_t *)(ws + p->lay.status);
    a.out = (__nv_bfloat16 *)out;
    a.k_new = (const unsigned char *)k_new;
    a.v_new = (const unsigned char *)v_new;
    a.touch = p->touch;
    a.touch_words = p->touch_words;
    a.head_mask = head_mask;
    a.tickets = (uint32_t *)(ws + p->lay.tickets);
    a.done = a.tickets + (size_t)kDecFusedMaxBatch * c.n_kv_heads;
    a.overlap = (p->launch_overlap && p->touch == nullptr) ? 1 : 0;   // the debug bitmap is written by the loaders
    a.key_begin = part ? part->key_begin : nullptr;
    a.key_end = part ? part->key_end : nullptr;
    a.pout_o = part ? part->out_o : nullptr;
    a.pout_ml = part ? part->out_ml : nullptr;
    a.push_world = part ? part->push.world : 0;
    a.push_rank = part ? part->push.rank : 0;
    a.push_seq = part ? part->push.seq : 0u;
    for (int i = 0; i < kMaxPeers; ++i) {
        const bool on = part && i < part->push.world;
        a.push_o[i] = on ? part->push.o[i] : nullptr;
        a.push_ml[i] = on ? part->push.ml[i] : nullptr;
        a.push_flags[i] = on ? part->push.flags[i] : nullptr;
    }
    a.push_ticket = (uint32_t *)(ws + p->lay.push_ticket);
    const int fused_max = p->decode_kernel == FLUX_DECODE_SINGLE_LAUNCH ? kDecFusedMaxBatch
                          : p->decode_kernel == FLUX_DECODE_AUTO        ? kDecFusedAutoBatch : 0;
    if (head_mask == nullptr && part == nullptr && B <= fused_max && c.n_kv_heads <= kDecFusedMaxKvHeads)
        return launch_decode_fused(p, a, st);
    const int rec = prof_begin(p, FLUX_KERNEL_DECODE, st);
    decode_kernel<<<p->dec_ctas, kDecWarps * 32, kDecSmemBytes, st>>>(a);
    prof_end(p, rec, st);
    p->launches++;
    int rc = check_cuda(cudaGetLastError(), "decode kernel launch");
    if (rc) return rc;
    decode_combine_kernel<<<B * c.n_q_heads, kCombWarps * 32, 0, st>>>(a);
    p->launches++;
    p->debug_records = B;
    return check_cuda(cudaGetLastError(), "decode combine kernel launch");
}

}  // namespace flux

// ---------------------------------------------------------------------------------------------
// Decode without any caller- or library-allocated scratch (flux_attn_decode_noalloc).
//
// Some callers have no way to obtain device memory for a workspace: a plug-in inside a host
// program that owns every byte of device memory and hands out only the tensors of the current
// operator, or a serving loop that must not meet the device-wide synchronisation an allocation
// can bring.  For them the split-K scratch (partials, schedule table, status word) lives in a
// fixed array inside the library image.  Every process that loads the library pays for it on
// every GPU it touches, so it is sized for moderate batches only.
// ---------------------------------------------------------------------------------------------
namespace flux {
namespace {

constexpr int kNaMaxBatch = 64;     // requests per call
constexpr int kNaMaxCtas = 160;     // CTAs launched (one per SM, clamped)
constexpr int kNaMaxG = 8;          // query heads per KV head
constexpr int kNaMaxHeadGroups = 2; // n_kv_heads <= 16
constexpr size_t kNaSlots = (size_t)(kNaMaxCtas + kNaMaxBatch * kNaMaxHeadGroups) * kDecWarps;
constexpr size_t kNaOffStatus = 0;
constexpr size_t kNaOffDebug = 256;
constexpr size_t kNaOffSched = kNaOffDebug + (size_t)kNaMaxBatch * 8 * sizeof(int32_t);
constexpr size_t kNaOffMl = (kNaOffSched + (kNaMaxBatch + 4) * sizeof(int32_t) + 255) / 256 * 256;
constexpr size_t kNaOffO = (kNaOffMl + kNaSlots * kNaMaxG * 2 * sizeof(float) + 255) / 256 * 256;
constexpr size_t kNaBytes = kNaOffO + kNaSlots * kNaMaxG * kHeadDim * sizeof(float);   // about 9.6 MB

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNaBytes];

struct NaDevice {
    bool ready;
    unsigned char *scratch;  // device address of g_noalloc_scratch on this device
    int n_ctas;
};
constexpr int kNaMaxDevices = 64;
NaDevice g_na_dev[kNaMaxDevices];
std::mutex g_na_mutex;

// Once per device, with that device current: resolve the scratch address, raise the kernel's
// dynamic shared-memory limit, read the SM count.
int noalloc_setup(int dev, NaDevice **out)
{
    if (dev < 0 || dev >= kNaMaxDevices) return fail(FLUX_E_CUDA, "device index %d not supported", dev);
    std::lock_guard<std::mutex> lock(g_na_mutex);
    NaDevice &d = g_na_dev[dev];
    if (!d.ready) {
        int major = 0, sms = 0, smem = 0;
        int rc = check_cuda(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev),
                            "cudaDeviceGetAttribute");
        if (!rc) rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev),
                                 "cudaDeviceGetAttribute");
        if (!rc) rc = check_cuda(cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev),
                                 "cudaDeviceGetAttribute");
        if (rc) return rc;
        if (major != 10) return fail(FLUX_E_CUDA, "this library is built for sm_100a only");
        if (smem < kDecSmemBytes) return fail(FLUX_E_CUDA, "not enough shared memory per block");
        void *ptr = nullptr;
        rc = check_cuda(cudaGetSymbolAddress(&ptr, g_noalloc_scratch), "cudaGetSymbolAddress(scratch)");
        if (rc) return rc;
        rc = check_cuda(cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kDecSmemBytes),
                        "cudaFuncSetAttribute(decode_kernel)");
        if (rc) return rc;
        d.scratch = (unsigned char *)ptr;
        d.n_ctas = sms < kNaMaxCtas ? sms : kNaMaxCtas;
        d.ready = true;
    }
    *out = &d;
    return FLUX_OK;
}

}  // namespace
}  // namespace flux

extern "C" int flux_attn_decode_noalloc(const flux_config *cfg, int32_t layer, int32_t B,
                                        const uint8_t *mask, const void *q,
                                        const void *const *k_caches, const void *const *v_caches,
                                        const int32_t *ctx_len, void *out, uint32_t *status_out,
                                        void *stream)
{
    using namespace flux;
    if (!cfg) return fail(FLUX_E_INVALID_ARG, "config is NULL");
    if (cfg->head_dim != kHeadDim) return fail(FLUX_E_UNSUPPORTED_SHAPE, "head_dim must be 128");
    if (cfg->n_layers < 1 || cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 ||
        cfg->n_q_heads % cfg->n_kv_heads != 0)
        return fail(FLUX_E_UNSUPPORTED_SHAPE, "bad head counts");
    if (cfg->sink < 0 || cfg->window < 1 || cfg->max_context < 1 ||
        (cfg->kv_layout != FLUX_KV_FULL && cfg->kv_layout != FLUX_KV_COMPACT_SA) ||
        !(cfg->softmax_scale >= 0.0f))
        return fail(FLUX_E_INVALID_ARG, "bad sink / window / max_context / kv_layout / softmax_scale");
    const int G = cfg->n_q_heads / cfg->n_kv_heads;
    const int n_hg = dec_head_groups(cfg->n_kv_heads);
    if (B < 1 || B > kNaMaxBatch)
        return fail(FLUX_E_CAPACITY, "flux_attn_decode_noalloc: B=%d exceeds the built-in scratch limit of %d "
                    "requests; use flux_attn_decode with a workspace", B, kNaMaxBatch);
    if (G > kNaMaxG || n_hg > kNaMaxHeadGroups)
        return fail(FLUX_E_CAPACITY, "flux_attn_decode_noalloc: %d query heads per KV head (limit %d) or %d KV "
                    "heads (limit 16) exceed the built-in scratch; use flux_attn_decode with a workspace",
                    G, kNaMaxG, cfg->n_kv_heads);
    if (layer < 0 || layer >= cfg->n_layers) return fail(FLUX_E_INVALID_ARG, "layer out of range");
    if (!mask || !q || !k_caches || !v_caches || !ctx_len || !out)
        return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    if ((((uintptr_t)q) | ((uintptr_t)out)) & 15u)
        return fail(FLUX_E_INVALID_ARG, "q / out must be 16-byte aligned");
    int dev = 0;
    int rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
    if (rc) return rc;
    NaDevice *nd = nullptr;
    rc = noalloc_setup(dev, &nd);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char *ws = nd->scratch;
    // the array keeps whatever the previous call left: the status word must start at zero
    rc = check_cuda(cudaMemsetAsync(ws + kNaOffStatus, 0, 256, st), "status clear");
    if (rc) return rc;
    DecArgs a;
    a.q = (const __nv_bfloat16 *)q;
    a.k_caches = k_caches;
    a.v_caches = v_caches;
    a.ctx_len = ctx_len;
    a.mask = mask;
    a.B = B; a.L = cfg->n_layers; a.layer = layer; a.Hq = cfg->n_q_heads; a.Hkv = cfg->n_kv_heads;
    a.G = G; a.S = cfg->sink; a.W = cfg->window; a.layout = cfg->kv_layout;
    a.max_context = cfg->max_context;
    const float scale = cfg->softmax_scale > 0.0f ? cfg->softmax_scale : 1.0f / sqrtf((float)kHeadDim);
    a.scale_log2 = scale * 1.4426950408889634f;
    a.part_o = (float *)(ws + kNaOffO);
    a.part_ml = (float *)(ws + kNaOffMl);
    a.debug = (int32_t *)(ws + kNaOffDebug);
    a.sched = (int32_t *)(ws + kNaOffSched);
    a.status = (uint32_t *)(ws + kNaOffStatus);
    a.out = (__nv_bfloat16 *)out;
    a.k_new = nullptr;
    a.v_new = nullptr;
    a.touch = nullptr;
    a.touch_words = 0;
    a.head_mask = nullptr;
    a.tickets = nullptr;
    a.done = nullptr;
    a.overlap = 0;
    a.key_begin = a.key_end = nullptr;
    a.pout_o = a.pout_ml = nullptr;
    a.push_world = 0;
    a.push_ticket = nullptr;
    decode_kernel<<<nd->n_ctas, kDecWarps * 32, kDecSmemBytes, st>>>(a);
    rc = check_cuda(cudaGetLastError(), "decode kernel launch");
    if (rc) return rc;
    decode_combine_kernel<<<B * cfg->n_q_heads, kCombWarps * 32, 0, st>>>(a);
    rc = check_cuda(cudaGetLastError(), "decode combine kernel launch");
    if (rc) return rc;
    if (status_out)
        rc = check_cuda(cudaMemcpyAsync(status_out, ws + kNaOffStatus, sizeof(uint32_t),
                                        cudaMemcpyDeviceToDevice, st), "status copy");
    return rc;
}
