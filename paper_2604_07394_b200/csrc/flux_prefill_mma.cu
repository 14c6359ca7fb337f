// Causal prefill of one routed layer with warp-level tensor-core MMAs (m16n8k16).
//
// One CTA = 64 query rows of one query head; it walks the KV tiles its rows keep:
// every tile up to the diagonal for an FA layer (Eq. 1), the sink tiles plus the
// window tiles for an SA layer (Eq. 2 with the streaming subset), so an SA layer
// costs O(N (S + W)).  Softmax is the online form in fp32; P is rounded to bf16
// for the PV product.  This kernel serves every shape (ragged tails, chunked
// prefill with q_start > 0, any sink / window); the tcgen05 kernel in
// flux_prefill_tc.cu takes over for the large aligned shapes.
#include "flux_internal.h"

namespace flux {
namespace {

constexpr int BM = 64, BN = 64, kWarps = 4;
constexpr int kTileBytes = BN * kRowBytes;                 // 16 KB
constexpr int kStages = 2;
constexpr int kSmemBytes = BM * kRowBytes + kStages * 2 * kTileBytes;  // Q + stages of (K, V)
constexpr float kNegBig = -1.0e30f;

struct PreArgs {
    const __nv_bfloat16 *q;
    const unsigned char *k;
    const unsigned char *v;
    __nv_bfloat16 *out;
    const uint8_t *mask;
    int L, layer, req, Hq, Hkv, G, S, W, q_start, Nq;
    float scale_log2;
    int32_t *debug;
    uint32_t *status;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

__global__ void __launch_bounds__(kWarps * 32) prefill_mma_kernel(PreArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t4 = lane & 3;
    const int n_qt = (a.Nq + BM - 1) / BM;
    const int qt = n_qt - 1 - blockIdx.x;  // heaviest (latest) tiles first
    const int h = blockIdx.y, kvh = h / a.G;
    const int q_end = a.q_start + a.Nq;    // also the number of KV rows present
    const int i0 = a.q_start + qt * BM;
    const int i_hi = min(i0 + BM - 1, q_end - 1);

    uint8_t mode_raw = a.mask[a.req * a.L + a.layer];
    if (mode_raw > 1 && tid == 0) atomicOr(a.status, FLUX_STATUS_BAD_MASK);
    const bool fa = mode_raw != 0;
    const int S = a.S, W = a.W;

    if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) {
        const int n = q_end;
        const bool two = !fa && n > S + W;
        int32_t *d = a.debug;
        d[0] = fa ? 1 : 0; d[1] = a.layer; d[2] = a.req; d[3] = n;
        d[4] = 0; d[5] = two ? S : n; d[6] = two ? n - W : 0; d[7] = two ? n : 0;
    }

    // KV tiles this query tile keeps: [0, e1) and [b2, e2)
    int e1, b2, e2 = i_hi / BN + 1;
    if (fa) {
        e1 = 0;
        b2 = 0;
    } else {
        e1 = min((S + BN - 1) / BN, e2);
        const int wb = max(0, i0 - W + 1);
        b2 = max(e1, wb / BN);
    }
    const int n_tiles = e1 + max(0, e2 - b2);

    unsigned char *sQ = smem;
    unsigned char *sKV = smem + BM * kRowBytes;
    const uint32_t sQ_u = smem_u32(sQ), sKV_u = smem_u32(sKV);

    const int lc = tid & 15, lr = tid >> 4;  // 16-byte chunk and first row of this thread's copies
    // Q tile
#pragma unroll
    for (int i = 0; i < BM / 8; ++i) {
        const int r = lr + 8 * i;
        const int row = i0 + r;
        const bool valid = row < q_end;
        const __nv_bfloat16 *src = a.q + ((size_t)(valid ? row - a.q_start : 0) * a.Hq + h) * kHeadDim + lc * 8;
        cp_async16(sQ_u + r * kRowBytes + ((lc ^ (r & 7)) << 4), src, valid ? 16 : 0);
    }
    auto issue = [&](int it, int stage) {
        const int jt = it < e1 ? it : b2 + (it - e1);
        const uint32_t kdst = sKV_u + stage * 2 * kTileBytes;
#pragma unroll
        for (int i = 0; i < BN / 8; ++i) {
            const int r = lr + 8 * i;
            const int j = jt * BN + r;
            const bool valid = j < q_end;
            const size_t off = ((size_t)(valid ? j : 0) * a.Hkv + kvh) * kRowBytes + lc * 16;
            const uint32_t dst = kdst + r * kRowBytes + ((lc ^ (r & 7)) << 4);
            cp_async16(dst, a.k + off, valid ? 16 : 0);
            cp_async16(dst + kTileBytes, a.v + off, valid ? 16 : 0);
        }
    };
    issue(0, 0);
    cp_async_commit();

    float o[16][4];
#pragma unroll
    for (int nt = 0; nt < 16; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[nt][e] = 0.f;
    float m_r[2] = {kNegBig, kNegBig}, l_r[2] = {0.f, 0.f};
    uint32_t qf[8][4];
    const int wr0 = warp * 16;
    const int mi = lane >> 3, rr = lane & 7;

    for (int it = 0; it < n_tiles; ++it) {
        if (it + 1 < n_tiles) {
            issue(it + 1, (it + 1) & 1);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        if (it == 0) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const int row = wr0 + (mi & 1) * 8 + rr;
                const int chunk = kk * 2 + (mi >> 1);
                ldmatrix_x4(qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3],
                            sQ_u + row * kRowBytes + ((chunk ^ rr) << 4));
            }
        }
        const int jt = it < e1 ? it : b2 + (it - e1);
        const int j0 = jt * BN;
        const uint32_t kb = sKV_u + (it & 1) * 2 * kTileBytes;
        const uint32_t vb = kb + kTileBytes;

        float s[8][4];
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) s[j][e] = 0.f;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
#pragma unroll
            for (int jp = 0; jp < 4; ++jp) {
                const int key = jp * 16 + (mi >> 1) * 8 + rr;
                const int chunk = kk * 2 + (mi & 1);
                uint32_t b0, b1, b2r, b3;
                ldmatrix_x4(b0, b1, b2r, b3, kb + key * kRowBytes + ((chunk ^ rr) << 4));
                mma_bf16(s[2 * jp], qf[kk], b0, b1);
                mma_bf16(s[2 * jp + 1], qf[kk], b2r, b3);
            }
        }
        // is every (row, key) pair of this tile kept?
        const int jmax = j0 + BN - 1;
        const bool full = (jmax <= i0) && (fa || jmax < S || j0 > i0 + BM - 1 - W);
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float x = s[j][e] * a.scale_log2;
                if (!full) {
                    const int key = j0 + j * 8 + 2 * t4 + (e & 1);
                    const int row = i0 + wr0 + g + 8 * (e >> 1);
                    const bool keep = key <= row && (fa || key < S || key > row - W);
                    x = keep ? x : -INFINITY;
                }
                s[j][e] = x;
            }
        float alpha[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 8; ++j) mx = fmaxf(mx, fmaxf(s[j][2 * i], s[j][2 * i + 1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_r[i], mx);
            alpha[i] = fast_exp2(m_r[i] - m_new);
            m_r[i] = m_new;
            float rs = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const float p = fast_exp2(s[j][2 * i + e] - m_new);
                    s[j][2 * i + e] = p;
                    rs += p;
                }
            l_r[i] = l_r[i] * alpha[i] + rs;
        }
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            o[nt][0] *= alpha[0];
            o[nt][1] *= alpha[0];
            o[nt][2] *= alpha[1];
            o[nt][3] *= alpha[1];
        }
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            uint32_t pa[4];
            pa[0] = pack_bf16(s[2 * ks][0], s[2 * ks][1]);
            pa[1] = pack_bf16(s[2 * ks][2], s[2 * ks][3]);
            pa[2] = pack_bf16(s[2 * ks + 1][0], s[2 * ks + 1][1]);
            pa[3] = pack_bf16(s[2 * ks + 1][2], s[2 * ks + 1][3]);
#pragma unroll
            for (int dt = 0; dt < 8; ++dt) {
                const int key = ks * 16 + (mi & 1) * 8 + rr;
                const int chunk = dt * 2 + (mi >> 1);
                uint32_t b0, b1, b2r, b3;
                ldmatrix_x4_trans(b0, b1, b2r, b3, vb + key * kRowBytes + ((chunk ^ rr) << 4));
                mma_bf16(o[2 * dt], pa, b0, b1);
                mma_bf16(o[2 * dt + 1], pa, b2r, b3);
            }
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 2; ++i) {
        l_r[i] += __shfl_xor_sync(0xffffffffu, l_r[i], 1);
        l_r[i] += __shfl_xor_sync(0xffffffffu, l_r[i], 2);
        const int row = i0 + wr0 + g + 8 * i;
        if (row < q_end) {
            const float inv = 1.f / l_r[i];
            __nv_bfloat16 *dst = a.out + ((size_t)(row - a.q_start) * a.Hq + h) * kHeadDim;
#pragma unroll
            for (int nt = 0; nt < 16; ++nt)
                *reinterpret_cast<uint32_t *>(dst + nt * 8 + 2 * t4) =
                    pack_bf16(o[nt][2 * i] * inv, o[nt][2 * i + 1] * inv);
        }
    }
}

}  // namespace

int prefill_mma_setup()
{
    return check_cuda(cudaFuncSetAttribute(prefill_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kSmemBytes),
                      "cudaFuncSetAttribute(prefill_mma_kernel)");
}

int launch_prefill_mma(flux_plan *p, int layer, int req, const void *q, const void *k, const void *v,
                       int q_start, int Nq, void *out, cudaStream_t st)
{
    const flux_config &c = p->cfg;
    char *ws = (char *)p->ws;
    PreArgs a;
    a.q = (const __nv_bfloat16 *)q;
    a.k = (const unsigned char *)k;
    a.v = (const unsigned char *)v;
    a.out = (__nv_bfloat16 *)out;
    a.mask = p->d_mask;
    a.L = c.n_layers; a.layer = layer; a.req = req; a.Hq = c.n_q_heads; a.Hkv = c.n_kv_heads;
    a.G = p->G; a.S = c.sink; a.W = c.window; a.q_start = q_start; a.Nq = Nq;
    a.scale_log2 = p->scale_log2;
    a.debug = (int32_t *)(ws + p->lay.debug);
    a.status = (uint32_t *)(ws + p->lay.status);
    dim3 grid((Nq + BM - 1) / BM, c.n_q_heads);
    const int rec = prof_begin(p, FLUX_KERNEL_PREFILL, st);
    prefill_mma_kernel<<<grid, kWarps * 32, kSmemBytes, st>>>(a);
    prof_end(p, rec, st);
    p->launches++;
    p->debug_records = 1;
    return check_cuda(cudaGetLastError(), "prefill kernel launch");
}

}  // namespace flux
