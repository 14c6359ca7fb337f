// Layer Router front end (Sec. 3.1, "Architecture and Feature Extraction"): Prefill-Suffix
// Pooling of the layer's query tensor over the first and the last prompt tokens (Appendix D.1:
// 100 + 100), a Context Encoder MLP and a Router Head MLP ending in the logits (pi_FA, pi_SA).
// The paper gives neither the pooling operator, the widths nor the activation; this file
// takes the token mean, Linear-SiLU-Linear for each MLP, and caller-chosen widths.
//
// The work is tiny and independent of the prompt length (at most 200 tokens of x_Q, a few MB of
// weights), so it is bound by launch and dependency latency, not by bandwidth.  One cooperative
// launch runs all five stages -- pooling, the four matrix-vector products -- with a grid-wide
// barrier (bounded spin on an arrival counter; the cooperative launch guarantees that every CTA
// is resident) between a stage and the next one that needs its whole output; the last stage,
// two rows, is done by the CTA that finishes the one before it last.  fp32 accumulation, bf16
// weights, deterministic reduction order.  Shapes whose largest activation vector does not fit
// the kernel's shared memory take five separate launches instead.
#include "flux_internal.h"
#include "flux_mma_util.h"
#include "flux_tc_util.h"

namespace flux {
namespace {

constexpr int kPoolCols = 64;       // bf16x2 columns per CTA
constexpr int kPoolGroups = 8;      // token groups per CTA (threadIdx.y)

// f[seg * F + c] = mean over the tokens of segment seg of x[token][c];  F = Hq * D (even).
// grid (F / 2 / kPoolCols, 2), block (kPoolCols, kPoolGroups).
__global__ void __launch_bounds__(kPoolCols *kPoolGroups)
router_pool_kernel(const __nv_bfloat162 *__restrict__ first, int n_first, const __nv_bfloat162 *__restrict__ last,
                   int n_last, float *__restrict__ f, int F2)
{
    __shared__ float2 part[kPoolGroups][kPoolCols];
    const int seg = blockIdx.y;
    const __nv_bfloat162 *x = seg ? last : first;
    const int n = seg ? n_last : n_first;
    const int col = blockIdx.x * kPoolCols + threadIdx.x;
    float2 acc = make_float2(0.f, 0.f);
    if (col < F2) {
#pragma unroll 4
        for (int t = threadIdx.y; t < n; t += kPoolGroups) {
            const float2 v = __bfloat1622float2(x[(size_t)t * F2 + col]);
            acc.x += v.x;
            acc.y += v.y;
        }
    }
    part[threadIdx.y][threadIdx.x] = acc;
    __syncthreads();
    if (threadIdx.y == 0 && col < F2) {
        float2 s = part[0][threadIdx.x];
#pragma unroll
        for (int g = 1; g < kPoolGroups; ++g) {
            s.x += part[g][threadIdx.x].x;
            s.y += part[g][threadIdx.x].y;
        }
        const float inv = 1.0f / (float)n;
        reinterpret_cast<float2 *>(f)[(size_t)seg * F2 + col] = make_float2(s.x * inv, s.y * inv);
    }
}

__device__ __forceinline__ float silu(float v) { return v / (1.0f + expf(-v)); }

// y = act(W x + b): W [n_out][n_in] bf16 row-major (n_in a multiple of 8, rows 16-byte aligned),
// x, b, y fp32.  One warp per output row; lanes stride over 16-byte pieces of the row, then a
// butterfly reduction.  A NaN / Inf result of the last layer is caught by the hard-routing kernel.
__global__ void __launch_bounds__(256)
router_linear_kernel(const __nv_bfloat16 *__restrict__ W, const float *__restrict__ b, const float *__restrict__ x,
                     float *__restrict__ y, int n_in, int n_out, int act)
{
    const int row = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    if (row >= n_out) return;
    const uint4 *w = reinterpret_cast<const uint4 *>(W + (size_t)row * n_in);
    const float4 *xv = reinterpret_cast<const float4 *>(x);
    float acc = 0.f;
    for (int i = lane; i < n_in / 8; i += 32) {
        const uint4 p = __ldg(w + i);
        const float4 x0 = xv[2 * i], x1 = xv[2 * i + 1];
        const float2 w0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.x));
        const float2 w1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.y));
        const float2 w2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.z));
        const float2 w3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.w));
        acc = fmaf(w0.x, x0.x, acc);
        acc = fmaf(w0.y, x0.y, acc);
        acc = fmaf(w1.x, x0.z, acc);
        acc = fmaf(w1.y, x0.w, acc);
        acc = fmaf(w2.x, x1.x, acc);
        acc = fmaf(w2.y, x1.y, acc);
        acc = fmaf(w3.x, x1.z, acc);
        acc = fmaf(w3.y, x1.w, acc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) {
        const float v = acc + b[row];
        y[row] = act ? silu(v) : v;
    }
}

int linear(const void *W, const float *b, const float *x, float *y, int n_in, int n_out, int act, cudaStream_t st)
{
    const int warps_per_cta = 8;
    router_linear_kernel<<<(n_out + warps_per_cta - 1) / warps_per_cta, warps_per_cta * 32, 0, st>>>(
        (const __nv_bfloat16 *)W, b, x, y, n_in, n_out, act);
    return check_cuda(cudaGetLastError(), "router linear kernel launch");
}


// ---- all stages in one cooperative launch ---------------------------------------------------

struct RouterArgs {
    const __nv_bfloat162 *first, *last;
    int n_first, n_last, F2;             // F2: bf16x2 columns of one token row (Hq * D / 2)
    const __nv_bfloat16 *w1, *w2, *w3, *w4;
    const float *b1, *b2, *b3, *b4;
    int F, E, R;
    float *f, *h1, *u, *h2, *logits;
    unsigned *sync;                      // [4]: three barrier counters, one ticket; zero between launches
    uint32_t *status;
    int xs_floats;                       // shared memory: the staged activation vector, then per warp pre_bytes of weight rows
    int pre_bytes, pre_off[3];           // byte offset of the prefetched row of stage 1 / 2 / 3 in a warp's area, -1: not prefetched
};

constexpr long long kRouterWaitCycles = 2000000000ll;   // bound of one barrier wait (about a second)

__device__ __forceinline__ unsigned ld_acquire(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Every CTA of the grid arrives; returns false when the wait ran out (flagged; the caller leaves).
__device__ __forceinline__ bool grid_barrier(unsigned *counter, uint32_t *status, int *s_abort)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;\n" ::"l"(counter) : "memory");
        const long long t0 = clock64();
        while (ld_acquire(counter) < gridDim.x) {
            if (clock64() - t0 > kRouterWaitCycles) {
                atomicOr(status, FLUX_STATUS_WAIT_EXPIRED);
                *s_abort = 1;
                break;
            }
        }
    }
    __syncthreads();
    return *s_abort == 0;
}

// One stage y = act(W x + b): x (written by other CTAs in this launch) is staged into shared memory, then
// one warp per output row, same order of operations as router_linear_kernel.  `pre`: this warp's first row,
// already brought into shared memory by the asynchronous copies issued at the start of the kernel (or NULL).
__device__ __forceinline__ void linear_stage(const __nv_bfloat16 *__restrict__ W, const float *__restrict__ b, const float *x,
                                             float *y, int n_in, int n_out, int act, float *xs, const unsigned char *pre)
{
    for (int i = threadIdx.x; i < n_in / 4; i += blockDim.x)
        reinterpret_cast<float4 *>(xs)[i] = __ldcg(reinterpret_cast<const float4 *>(x) + i);
    __syncthreads();
    const int lane = threadIdx.x & 31, warps = (int)(gridDim.x * blockDim.x) >> 5;
    const float4 *xv = reinterpret_cast<const float4 *>(xs);
    const int row0 = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    for (int row = row0; row < n_out; row += warps) {
        const bool staged = pre != nullptr && row == row0;
        const uint4 *w = staged ? reinterpret_cast<const uint4 *>(pre) : reinterpret_cast<const uint4 *>(W + (size_t)row * n_in);
        // four independent partial sums per lane (one per pair of weights of a 16-byte piece), added in a fixed order
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 4
        for (int i = lane; i < n_in / 8; i += 32) {
            const uint4 p = staged ? w[i] : __ldg(w + i);
            const float4 x0 = xv[2 * i], x1 = xv[2 * i + 1];
            const float2 w0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.x));
            const float2 w1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.y));
            const float2 w2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.z));
            const float2 w3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.w));
            a0 = fmaf(w0.y, x0.y, fmaf(w0.x, x0.x, a0));
            a1 = fmaf(w1.y, x0.w, fmaf(w1.x, x0.z, a1));
            a2 = fmaf(w2.y, x1.y, fmaf(w2.x, x1.x, a2));
            a3 = fmaf(w3.y, x1.w, fmaf(w3.x, x1.z, a3));
        }
        float acc = (a0 + a1) + (a2 + a3);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) {
            const float v = acc + b[row];
            y[row] = act ? silu(v) : v;
        }
    }
}

__global__ void __launch_bounds__(256) router_fused_kernel(RouterArgs a)
{
    extern __shared__ __align__(16) float xs[];
    __shared__ float2 part[8][32];
    __shared__ int s_abort;
    __shared__ unsigned s_ticket;
    __shared__ __align__(8) unsigned long long s_bar[3];   // weight rows of stage 1 / 2 / 3 have landed
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) s_abort = 0;
    // ---- the weights do not depend on anything computed here: every warp requests the first row it will need in
    //      each stage right away (one group of asynchronous copies per stage), so the 21 MB are in flight while the
    //      pooling and the first barrier run ----
    unsigned char *pre = reinterpret_cast<unsigned char *>(xs + a.xs_floats) + (size_t)warp * a.pre_bytes;
    const uint32_t bar0 = smem_u32(s_bar);
    if (tid == 0) {
        for (int s = 0; s < 3; ++s) tc::mbar_init(bar0 + 8 * s, 8);           // one arrival per warp
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (lane == 0) {
        const int row0 = (int)((blockIdx.x * blockDim.x + tid) >> 5);
        const __nv_bfloat16 *Ws[3] = {a.w1, a.w2, a.w3};
        const int n_in[3] = {a.F, a.E, a.E}, n_out[3] = {a.E, a.E, a.R};
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            if (a.pre_off[s] >= 0 && row0 < n_out[s]) {       // one bulk copy per row: n_in * 2 bytes, 16-byte aligned
                const uint32_t bytes = (uint32_t)n_in[s] * 2u;
                tc::mbar_expect_tx(bar0 + 8 * s, bytes);
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                             ::"r"(smem_u32(pre + a.pre_off[s])), "l"(Ws[s] + (size_t)row0 * n_in[s]), "r"(bytes), "r"(bar0 + 8 * s)
                             : "memory");
            } else {
                tc::mbar_arrive(bar0 + 8 * s);
            }
        }
    }
    // ---- pooling: a CTA takes 32 bf16x2 columns of one segment at a time; warp w sums tokens w, w + 8, ... ----
    const int slabs = (a.F2 + 31) / 32;
    for (int item = blockIdx.x; item < 2 * slabs; item += gridDim.x) {
        const int seg = item / slabs, col = (item % slabs) * 32 + lane;
        const __nv_bfloat162 *x = seg ? a.last : a.first;
        const int n = seg ? a.n_last : a.n_first;
        float2 acc = make_float2(0.f, 0.f);
        if (col < a.F2) {
#pragma unroll 8
            for (int t = warp; t < n; t += 8) {
                const float2 v = __bfloat1622float2(x[(size_t)t * a.F2 + col]);
                acc.x += v.x;
                acc.y += v.y;
            }
        }
        __syncthreads();      // the previous item's sums have been read
        part[warp][lane] = acc;
        __syncthreads();
        if (warp == 0 && col < a.F2) {
            float2 sum = part[0][lane];
#pragma unroll
            for (int g = 1; g < 8; ++g) {
                sum.x += part[g][lane].x;
                sum.y += part[g][lane].y;
            }
            const float inv = 1.0f / (float)n;
            reinterpret_cast<float2 *>(a.f)[(size_t)seg * a.F2 + col] = make_float2(sum.x * inv, sum.y * inv);
        }
    }
    // A CTA that gives up at a barrier still has copies in flight into its shared memory: it waits for them first
    // (bounded: the weights' arrival does not depend on any other CTA).
    auto rows_landed = [&](int s) -> bool {
        bool ok = tc::mbar_try(bar0 + 8 * s, 0u);
        for (const long long t0 = clock64(); !ok && clock64() - t0 < kRouterWaitCycles;) ok = tc::mbar_try(bar0 + 8 * s, 0u);
        if (!ok) {
            atomicOr(a.status, FLUX_STATUS_WAIT_EXPIRED);
            s_abort = 1;
        }
        return __all_sync(0xffffffffu, ok);
    };
    auto leave = [&]() { for (int s = 0; s < 3; ++s) rows_landed(s); };
    if (!grid_barrier(a.sync + 0, a.status, &s_abort)) { leave(); return; }
    if (!rows_landed(0)) { leave(); return; }
    linear_stage(a.w1, a.b1, a.f, a.h1, a.F, a.E, 1, xs, a.pre_off[0] >= 0 ? pre + a.pre_off[0] : nullptr);
    if (!grid_barrier(a.sync + 1, a.status, &s_abort)) { leave(); return; }
    if (!rows_landed(1)) { leave(); return; }
    linear_stage(a.w2, a.b2, a.h1, a.u, a.E, a.E, 0, xs, a.pre_off[1] >= 0 ? pre + a.pre_off[1] : nullptr);
    if (!grid_barrier(a.sync + 2, a.status, &s_abort)) { leave(); return; }
    if (!rows_landed(2)) { leave(); return; }
    linear_stage(a.w3, a.b3, a.u, a.h2, a.E, a.R, 1, xs, a.pre_off[2] >= 0 ? pre + a.pre_off[2] : nullptr);
    // ---- the two logits: by the CTA that finishes the stage above last ----
    __syncthreads();
    if (tid == 0) {
        unsigned ticket;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;\n" : "=r"(ticket) : "l"(a.sync + 3) : "memory");
        s_ticket = ticket;
    }
    __syncthreads();
    if (s_ticket != gridDim.x - 1) return;
    if (warp < 2) {
        const uint4 *w = reinterpret_cast<const uint4 *>(a.w4 + (size_t)warp * a.R);
        const float4 *xv = reinterpret_cast<const float4 *>(a.h2);
        float acc = 0.f;
        for (int i = lane; i < a.R / 8; i += 32) {
            const uint4 p = __ldg(w + i);
            const float4 x0 = __ldcg(xv + 2 * i), x1 = __ldcg(xv + 2 * i + 1);
            const float2 w0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.x));
            const float2 w1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.y));
            const float2 w2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.z));
            const float2 w3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.w));
            acc = fmaf(w0.x, x0.x, acc);
            acc = fmaf(w0.y, x0.y, acc);
            acc = fmaf(w1.x, x0.z, acc);
            acc = fmaf(w1.y, x0.w, acc);
            acc = fmaf(w2.x, x1.x, acc);
            acc = fmaf(w2.y, x1.y, acc);
            acc = fmaf(w3.x, x1.z, acc);
            acc = fmaf(w3.y, x1.w, acc);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) a.logits[warp] = acc + a.b4[warp];
    }
    if (tid < 4) a.sync[tid] = 0u;   // ready for the next launch (every other CTA is past all of them)
}

constexpr int kRouterFusedMaxFloats = 48 * 1024;   // largest activation vector staged in shared memory (192 KB)
constexpr int kRouterSmemLimit = 227 * 1024 - 2304;   // dynamic shared memory the kernel may ask for (its static part is about 2 KB)

}  // namespace

int router_setup(flux_plan *p)
{
    return check_cuda(cudaFuncSetAttribute(router_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kRouterSmemLimit),
                      "cudaFuncSetAttribute(router_fused_kernel)");
}

int launch_router_frontend(flux_plan *p, const flux_router_weights *w, const void *q_first, int n_first,
                           const void *q_last, int n_last, float *d_logits_out, cudaStream_t st)
{
    const int F1 = p->cfg.n_q_heads * kHeadDim, F = 2 * F1, E = w->enc_dim, R = w->head_hidden;
    float *scr = (float *)((char *)p->ws + p->lay.router);
    float *f = scr, *h1 = f + F, *u = h1 + kRouterMaxWidth, *h2 = u + kRouterMaxWidth;
    const int widest = F > E ? (F > R ? F : R) : (E > R ? E : R);
    if (widest <= kRouterFusedMaxFloats) {
        RouterArgs a;
        a.first = (const __nv_bfloat162 *)q_first; a.last = (const __nv_bfloat162 *)q_last;
        a.n_first = n_first; a.n_last = n_last; a.F2 = F1 / 2;
        a.w1 = (const __nv_bfloat16 *)w->w_enc1; a.w2 = (const __nv_bfloat16 *)w->w_enc2;
        a.w3 = (const __nv_bfloat16 *)w->w_head1; a.w4 = (const __nv_bfloat16 *)w->w_head2;
        a.b1 = w->b_enc1; a.b2 = w->b_enc2; a.b3 = w->b_head1; a.b4 = w->b_head2;
        a.F = F; a.E = E; a.R = R;
        a.f = f; a.h1 = h1; a.u = u; a.h2 = h2; a.logits = d_logits_out;
        a.sync = (unsigned *)((char *)p->ws + p->lay.router_sync);
        a.status = (uint32_t *)((char *)p->ws + p->lay.status);
        // shared memory: the widest activation vector, then per warp the weight rows requested ahead (as many
        // stages as fit, the first stage -- by far the largest -- first)
        a.xs_floats = widest;
        const int row_bytes[3] = {F * 2, E * 2, E * 2};
        int used = 0;
        for (int s = 0; s < 3; ++s) {
            a.pre_off[s] = -1;
            if ((size_t)widest * sizeof(float) + 8 * (size_t)(used + row_bytes[s]) <= (size_t)kRouterSmemLimit) {
                a.pre_off[s] = used;
                used += row_bytes[s];
            }
        }
        a.pre_bytes = used;
        const size_t smem = (size_t)widest * sizeof(float) + 8 * (size_t)used;
        void *args[] = {&a};
        // a cooperative launch either has every CTA resident (what the barriers need) or fails
        int rc = check_cuda(cudaLaunchCooperativeKernel((const void *)router_fused_kernel, dim3((unsigned)p->dev.n_sms), dim3(256),
                                                        args, smem, st),
                            "router kernel launch");
        if (rc) return rc;
        p->launches += 1;
        return FLUX_OK;
    }
    const dim3 grid((F1 / 2 + kPoolCols - 1) / kPoolCols, 2), block(kPoolCols, kPoolGroups);
    router_pool_kernel<<<grid, block, 0, st>>>((const __nv_bfloat162 *)q_first, n_first, (const __nv_bfloat162 *)q_last,
                                               n_last, f, F1 / 2);
    int rc = check_cuda(cudaGetLastError(), "router pooling kernel launch");
    if (rc) return rc;
    if ((rc = linear(w->w_enc1, w->b_enc1, f, h1, F, E, 1, st))) return rc;
    if ((rc = linear(w->w_enc2, w->b_enc2, h1, u, E, E, 0, st))) return rc;
    if ((rc = linear(w->w_head1, w->b_head1, u, h2, E, R, 1, st))) return rc;
    if ((rc = linear(w->w_head2, w->b_head2, h2, d_logits_out, R, 2, 0, st))) return rc;
    p->launches += 5;
    return FLUX_OK;
}

}  // namespace flux
