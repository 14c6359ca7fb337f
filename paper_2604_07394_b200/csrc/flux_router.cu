// Layer Router front end (Sec. 3.1, "Architecture and Feature Extraction"): Prefill-Suffix
// Pooling of the layer's query tensor over the first and the last prompt tokens (Appendix D.1:
// 100 + 100), a Context Encoder MLP and a Router Head MLP ending in the logits (pi_FA, pi_SA).
// The paper gives neither the pooling operator, the widths nor the activation; this file
// takes the token mean, Linear-SiLU-Linear for each MLP, and caller-chosen widths.
//
// The work is tiny and independent of the prompt length (at most 200 tokens of x_Q, a few MB of
// weights), so it is bound by launch and dependency latency, not by bandwidth.  One launch of one
// CTA per SM runs all five stages -- pooling, the four matrix-vector products.  The pooled
// descriptor is handed to the first product through a grid-wide barrier (bounded spin on an
// arrival counter; a grid of one CTA per SM is resident as soon as the kernel before it has
// left).  The later activations are small, so each value travels with a tag -- the launch's
// number -- in one 64-bit word, and a consumer simply re-reads its inputs until their tags are
// this launch's: one trip to L2 after the producer's store instead of a barrier plus a read.
// The launch allows programmatic overlap with the kernel before it in the stream: the weight
// rows are requested while that kernel drains.  fp32 accumulation, bf16 weights, deterministic
// reduction order.
#include "flux_internal.h"
#include "flux_mma_util.h"
#include "flux_tc_util.h"

namespace flux {
namespace {

__device__ __forceinline__ float silu(float v) { return v / (1.0f + expf(-v)); }

// Weights W [n_out][n_in] are bf16 row-major with n_in a multiple of 8 (rows 16-byte aligned); activations,
// biases and results are fp32.  A NaN / Inf logit is caught by the hard-routing kernel.

struct RouterArgs {
    const __nv_bfloat162 *first, *last;
    int n_first, n_last, F2;             // F2: bf16x2 columns of one token row (Hq * D / 2)
    const __nv_bfloat16 *w1, *w2, *w3, *w4;
    const float *b1, *b2, *b3, *b4;
    int F, E, R;
    float *f, *logits;
    unsigned long long *h1, *u, *h2;     // tagged activations: low word the fp32 value, high word the launch number
    unsigned *sync;                      // [0] barrier counter, [1] exit ticket (both zero between launches), [2] last launch number
    uint32_t *status;
    int pre_bytes, pre_off[3];           // shared memory: eight areas of pre_bytes, one per output row of a CTA's first pass;
                                         // byte offset of the row of stage 1 / 2 / 3 in an area, -1: not brought in ahead
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

constexpr int kRouterWarps = 16;

// One stage y = act(W x + b) for the CTA's output rows, eight at a time.  The input vector is cut into 16-byte pieces
// of weights (eight inputs); warp w takes the pieces 32 (w + 16 j) .. 32 (w + 16 j) + 31, one per lane, reads their
// eight inputs once (through L2 only: other SMs wrote them) and multiplies them into all eight rows, so a row of
// weights and the input vector are each read once per CTA.  fp32 FMAs in a fixed order; per row a butterfly over the
// lanes, then the sixteen warps' sums added in warp order.  `pre`: the CTA's first eight rows (row r at
// pre + r * pre_stride), brought into shared memory by the bulk copies issued at the start of the kernel, or NULL.
__device__ __forceinline__ void st_tagged(unsigned long long *p, float v, unsigned epoch)
{
    const unsigned long long w = ((unsigned long long)epoch << 32) | (unsigned long long)__float_as_uint(v);
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;\n" ::"l"(p), "l"(w) : "memory");
}

// The eight tagged inputs of piece i, re-read until every tag is this launch's.  false: the wait ran out.
__device__ __forceinline__ bool ld_tagged_piece(const unsigned long long *x, int i, unsigned epoch, float4 &x0, float4 &x1)
{
    unsigned long long w[8];
    long long t0 = 0;
    for (;;) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
            asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];\n" : "=l"(w[2 * k]), "=l"(w[2 * k + 1]) : "l"(x + 8 * (size_t)i + 2 * k) : "memory");
        bool ok = true;
#pragma unroll
        for (int k = 0; k < 8; ++k) ok = ok && (unsigned)(w[k] >> 32) == epoch;
        if (ok) break;
        if (t0 == 0) t0 = clock64();
        else if (clock64() - t0 > kRouterWaitCycles) return false;
    }
    x0 = make_float4(__uint_as_float((unsigned)w[0]), __uint_as_float((unsigned)w[1]), __uint_as_float((unsigned)w[2]), __uint_as_float((unsigned)w[3]));
    x1 = make_float4(__uint_as_float((unsigned)w[4]), __uint_as_float((unsigned)w[5]), __uint_as_float((unsigned)w[6]), __uint_as_float((unsigned)w[7]));
    return true;
}

__device__ __forceinline__ void accumulate_piece(float (&acc)[8][2], const uint4 p, const float4 x0, const float4 x1, int r)
{
    const float2 w0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.x));
    const float2 w1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.y));
    const float2 w2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.z));
    const float2 w3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&p.w));
    acc[r][0] = fmaf(w1.y, x0.w, fmaf(w1.x, x0.z, fmaf(w0.y, x0.y, fmaf(w0.x, x0.x, acc[r][0]))));
    acc[r][1] = fmaf(w3.y, x1.w, fmaf(w3.x, x1.z, fmaf(w2.y, x1.y, fmaf(w2.x, x1.x, acc[r][1]))));
}

// x_plain: the input as plain floats (complete: a grid-wide barrier came before); else x_tagged.  The output is
// tagged.  `bias0`: b[row] of the first pass for threads 0..7, read at the start of the kernel (a late read would put
// one more trip to memory on the critical path).  false: a wait ran out (flagged), the caller leaves.
__device__ __forceinline__ bool linear_stage(const __nv_bfloat16 *__restrict__ W, const float *__restrict__ b, const float *x_plain,
                                             const unsigned long long *x_tagged, unsigned long long *y, int n_in, int n_out,
                                             int act, const unsigned char *pre, size_t pre_stride, float bias0, unsigned epoch,
                                             float (*s_part)[8], int *s_abort, uint32_t *status)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_pieces = n_in / 8;
    const int base0 = (int)blockIdx.x * 8;
    for (int base = base0; base < n_out; base += (int)gridDim.x * 8) {
        const bool staged = pre != nullptr && base == base0;   // rows in shared memory (rows beyond n_out were not copied and are skipped)
        float acc[8][2];
#pragma unroll
        for (int r = 0; r < 8; ++r) acc[r][0] = acc[r][1] = 0.f;
        for (int i = warp * 32 + lane; i < n_pieces; i += kRouterWarps * 32) {
            float4 x0, x1;
            if (x_plain) {
                x0 = __ldcg(reinterpret_cast<const float4 *>(x_plain) + 2 * i);
                x1 = __ldcg(reinterpret_cast<const float4 *>(x_plain) + 2 * i + 1);
            } else if (!ld_tagged_piece(x_tagged, i, epoch, x0, x1)) {
                atomicOr(status, FLUX_STATUS_WAIT_EXPIRED);
                *reinterpret_cast<volatile int *>(s_abort) = 1;
                break;
            }
            if (staged) {
#pragma unroll
                for (int r = 0; r < 8; ++r)
                    if (base + r < n_out) accumulate_piece(acc, reinterpret_cast<const uint4 *>(pre + r * pre_stride)[i], x0, x1, r);
            } else {
#pragma unroll
                for (int r = 0; r < 8; ++r)
                    if (base + r < n_out)
                        accumulate_piece(acc, __ldg(reinterpret_cast<const uint4 *>(W + (size_t)(base + r) * n_in) + i), x0, x1, r);
            }
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            float v = acc[r][0] + acc[r][1];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0) s_part[warp][r] = v;
        }
        __syncthreads();
        if (*reinterpret_cast<volatile int *>(s_abort)) return false;
        if (threadIdx.x < 8 && base + (int)threadIdx.x < n_out) {
            float v = s_part[0][threadIdx.x];
#pragma unroll
            for (int w = 1; w < kRouterWarps; ++w) v += s_part[w][threadIdx.x];
            v += base == base0 ? bias0 : b[base + threadIdx.x];
            st_tagged(y + base + threadIdx.x, act ? silu(v) : v, epoch);
        }
        __syncthreads();
    }
    return true;
}

constexpr int kRouterThreads = kRouterWarps * 32;
constexpr int kRouterLastEarly = 2;   // 16-byte pieces per lane of a last-stage row read at the start (covers a head width of 512)

__global__ void __launch_bounds__(kRouterThreads) router_fused_kernel(RouterArgs a)
{
    extern __shared__ __align__(16) unsigned char rows[];
    __shared__ float2 part[kRouterWarps][32];
    __shared__ float s_part[kRouterWarps][8];
    __shared__ int s_abort;
    __shared__ __align__(8) unsigned long long s_bar[3];   // weight rows of stage 1 / 2 / 3 have landed
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // The launch is issued with programmatic stream serialisation: dependents are released at once, and the weights
    // -- constants of the model, which the previous kernel in the stream does not write -- are requested before the
    // grid-dependency wait: every CTA asks for the first eight rows it will need in each stage (one bulk copy per row
    // onto an mbarrier per stage), so the 21 MB are in flight while the previous launch drains and while the pooling
    // and the first barrier run.  Everything else (the x_Q tokens, the activations, the counters) comes after the wait.
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    if (tid == 0) s_abort = 0;
    unsigned char *pre = rows + (size_t)(warp & 7) * a.pre_bytes;
    const uint32_t bar0 = smem_u32(s_bar);
    if (tid == 0) {
        for (int s = 0; s < 3; ++s) tc::mbar_init(bar0 + 8 * s, 8);           // one arrival per row slot
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (lane == 0 && warp < 8) {
        const int row0 = (int)blockIdx.x * 8 + warp;
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
    // constants that sit on the critical path later: the biases of this CTA's first rows and, in the last CTA (which
    // has the fewest rows and computes the logits), the two rows of the last stage
    float bias0[3] = {0.f, 0.f, 0.f};
    if (tid < 8) {
        const int row0 = (int)blockIdx.x * 8 + tid;
        if (row0 < a.E) bias0[0] = __ldg(a.b1 + row0), bias0[1] = __ldg(a.b2 + row0);
        if (row0 < a.R) bias0[2] = __ldg(a.b3 + row0);
    }
    uint4 w4_early[kRouterLastEarly];
    float b4_early = 0.f;
    const bool does_logits = blockIdx.x == gridDim.x - 1;
    if (does_logits && warp < 2) {
#pragma unroll
        for (int j = 0; j < kRouterLastEarly; ++j) {
            const int i = lane + 32 * j;
            w4_early[j] = i < a.R / 8 ? __ldg(reinterpret_cast<const uint4 *>(a.w4 + (size_t)warp * a.R) + i) : make_uint4(0u, 0u, 0u, 0u);
        }
        b4_early = __ldg(a.b4 + warp);
    }
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    unsigned epoch = __ldcg(a.sync + 2) + 1u;      // this launch's number (the one before it has finished and stored its own)
    if (epoch == 0u) epoch = 1u;                    // zero is what a cleared buffer holds
    // ---- pooling: a CTA takes 32 bf16x2 columns of one segment at a time; warp w sums tokens w, w + kRouterWarps, ... (in that order) ----
    const int slabs = (a.F2 + 31) / 32;
    for (int item = blockIdx.x; item < 2 * slabs; item += gridDim.x) {
        const int seg = item / slabs, col = (item % slabs) * 32 + lane;
        const __nv_bfloat162 *x = seg ? a.last : a.first;
        const int n = seg ? a.n_last : a.n_first;
        float2 acc = make_float2(0.f, 0.f);
        if (col < a.F2) {
            // eight loads in flight per lane (a loop with a data-dependent trip count would take them one by one)
            for (int t0 = warp; t0 < n; t0 += 8 * kRouterWarps) {
                __nv_bfloat162 v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int t = t0 + j * kRouterWarps;
                    v[j] = t < n ? x[(size_t)t * a.F2 + col] : __float2bfloat162_rn(0.f);
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float2 f2 = __bfloat1622float2(v[j]);
                    acc.x += f2.x;
                    acc.y += f2.y;
                }
            }
        }
        __syncthreads();      // the previous item's sums have been read
        part[warp][lane] = acc;
        __syncthreads();
        if (warp == 0 && col < a.F2) {
            float2 sum = part[0][lane];
#pragma unroll
            for (int g = 1; g < kRouterWarps; ++g) {
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
    if (!linear_stage(a.w1, a.b1, a.f, nullptr, a.h1, a.F, a.E, 1, a.pre_off[0] >= 0 ? rows + a.pre_off[0] : nullptr,
                      (size_t)a.pre_bytes, bias0[0], epoch, s_part, &s_abort, a.status)) { leave(); return; }
    if (!rows_landed(1)) { leave(); return; }
    if (!linear_stage(a.w2, a.b2, nullptr, a.h1, a.u, a.E, a.E, 0, a.pre_off[1] >= 0 ? rows + a.pre_off[1] : nullptr,
                      (size_t)a.pre_bytes, bias0[1], epoch, s_part, &s_abort, a.status)) { leave(); return; }
    if (!rows_landed(2)) { leave(); return; }
    if (!linear_stage(a.w3, a.b3, nullptr, a.u, a.h2, a.E, a.R, 1, a.pre_off[2] >= 0 ? rows + a.pre_off[2] : nullptr,
                      (size_t)a.pre_bytes, bias0[2], epoch, s_part, &s_abort, a.status)) { leave(); return; }
    // ---- the two logits ----
    if (does_logits && warp < 2) {
        const uint4 *w = reinterpret_cast<const uint4 *>(a.w4 + (size_t)warp * a.R);
        float acc = 0.f;
        bool ok = true;
        auto piece = [&](const uint4 p, int i) {
            float4 x0, x1;
            if (!ld_tagged_piece(a.h2, i, epoch, x0, x1)) { ok = false; return; }
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
        };
#pragma unroll
        for (int j = 0; j < kRouterLastEarly; ++j)
            if (lane + 32 * j < a.R / 8) piece(w4_early[j], lane + 32 * j);
        for (int i = lane + 32 * kRouterLastEarly; i < a.R / 8 && ok; i += 32) piece(__ldg(w + i), i);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (!__all_sync(0xffffffffu, ok)) {
            if (lane == 0) atomicOr(a.status, FLUX_STATUS_WAIT_EXPIRED);
        } else if (lane == 0) {
            a.logits[warp] = acc + b4_early;
        }
    }
    // ---- the CTA that leaves last puts the counters back and records the launch number ----
    __syncthreads();
    if (tid == 0) {
        unsigned ticket;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;\n" : "=r"(ticket) : "l"(a.sync + 1) : "memory");
        if (ticket == gridDim.x - 1) {
            a.sync[0] = 0u;
            a.sync[1] = 0u;
            a.sync[2] = epoch;
        }
    }
}

constexpr int kRouterSmemLimit = 227 * 1024 - 5120;   // dynamic shared memory the kernel may ask for (its static part is about 4.6 KB)

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
    float *f = scr;
    unsigned long long *h1 = reinterpret_cast<unsigned long long *>(f + F), *u = h1 + kRouterMaxWidth, *h2 = u + kRouterMaxWidth;
    {
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
        // shared memory: per output row of a CTA's first pass, the weight rows requested ahead (as many stages as
        // fit, the first stage -- by far the largest -- first)
        const int row_bytes[3] = {F * 2, E * 2, E * 2};
        int used = 0;
        for (int s = 0; s < 3; ++s) {
            a.pre_off[s] = -1;
            if (8 * (size_t)(used + row_bytes[s]) <= (size_t)kRouterSmemLimit) {
                a.pre_off[s] = used;
                used += row_bytes[s];
            }
        }
        a.pre_bytes = used;
        const size_t smem = 8 * (size_t)used;
        // One CTA per SM: the grid-wide barriers need every CTA resident, which a grid of that size is as soon as the
        // previous kernel's CTAs have left (the launch may start while they drain; see the kernel).
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3((unsigned)p->dev.n_sms);
        lc.blockDim = dim3(kRouterThreads);
        lc.dynamicSmemBytes = smem;
        lc.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = attr;
        lc.numAttrs = 1;
        int rc = check_cuda(cudaLaunchKernelEx(&lc, router_fused_kernel, a), "router kernel launch");
        if (rc) return rc;
        p->launches += 1;
        return FLUX_OK;
    }
}

}  // namespace flux
