// Layer Router front end (Sec. 3.1, "Architecture and Feature Extraction"): Prefill-Suffix
// Pooling of the layer's query tensor over the first and the last prompt tokens (Appendix D.1:
// 100 + 100), a Context Encoder MLP and a Router Head MLP ending in the logits (pi_FA, pi_SA).
// The paper gives neither the pooling operator, the widths nor the activation; this file
// takes the token mean, Linear-SiLU-Linear for each MLP, and caller-chosen widths.
//
// The work is tiny and independent of the prompt length (at most 200 tokens of x_Q, a few MB of
// weights): one pooling launch and four matrix-vector launches, all HBM / latency bound; fp32
// accumulation, bf16 weights, deterministic reduction order.
#include "flux_internal.h"

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

}  // namespace

int launch_router_frontend(flux_plan *p, const flux_router_weights *w, const void *q_first, int n_first,
                           const void *q_last, int n_last, float *d_logits_out, cudaStream_t st)
{
    const int F1 = p->cfg.n_q_heads * kHeadDim, F = 2 * F1, E = w->enc_dim, R = w->head_hidden;
    float *scr = (float *)((char *)p->ws + p->lay.router);
    float *f = scr, *h1 = f + F, *u = h1 + kRouterMaxWidth, *h2 = u + kRouterMaxWidth;
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
