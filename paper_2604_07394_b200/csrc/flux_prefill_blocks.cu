// Causal prefill under a block mask (block size 64) with warp-level tensor-core MMAs (m16n8k16).
//
// Sparse Attention, Eq. 2, with the condensed subset given block by block: the sparse kernels
// the paper runs select keys in 64 x 64 blocks (Appendix D.3, "block size ... the minimum unit
// of sparsity"), which covers its streaming pattern at block granularity and patterns that pick
// blocks by score.  One CTA = one query block (64 rows) of one query head; it compacts its row
// of the mask into a list of kept key blocks in shared memory and walks only those, with
// elementwise causal masking on the diagonal block alone.  Softmax is the online form in fp32;
// P is rounded to bf16 for the PV product.
#include "flux_internal.h"

namespace flux {
namespace {

constexpr int BM = 64, BN = 64, kWarps = 4;
constexpr int kTileBytes = BN * kRowBytes;                 // 16 KB
constexpr int kStages = 2;
constexpr int kMaxKvBlocks = 4096;                         // 256K positions
constexpr int kListOff = BM * kRowBytes + kStages * 2 * kTileBytes;   // Q + stages of (K, V), then the block list
constexpr int kSmemBytes = kListOff + kMaxKvBlocks * 2;
constexpr float kNegBig = -1.0e30f;

struct BlkArgs {
    const __nv_bfloat16 *q;
    const unsigned char *k;
    const unsigned char *v;
    __nv_bfloat16 *out;
    const uint8_t *bm;          // [query block (absolute)][n_kb]
    int n_kb, Hq, Hkv, G, q_start, Nq;
    float scale_log2;
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

__global__ void __launch_bounds__(kWarps * 32) prefill_blocks_kernel(BlkArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t4 = lane & 3;
    const int n_qt = (a.Nq + BM - 1) / BM;
    const int qt = n_qt - 1 - blockIdx.x;  // heaviest (latest) blocks first for dense masks
    const int h = blockIdx.y, kvh = h / a.G;
    const int q_end = a.q_start + a.Nq;    // also the number of KV rows present
    const int i0 = a.q_start + qt * BM;
    const int qb = i0 / BM;                // absolute query block

    // kept key blocks of this query block, in order, as a list in shared memory
    uint16_t *list = reinterpret_cast<uint16_t *>(smem + kListOff);
    __shared__ int s_count;
    if (warp == 0) {
        const uint8_t *row = a.bm + (size_t)qb * a.n_kb;
        const int last = min(qb, a.n_kb - 1);       // causality: nothing beyond the diagonal block
        int cnt = 0;
        for (int base = 0; base <= last; base += 32) {
            const int kb = base + lane;
            const bool keep = kb <= last && row[kb] != 0;
            const unsigned bal = __ballot_sync(0xffffffffu, keep);
            if (keep) list[cnt + __popc(bal & ((1u << lane) - 1u))] = (uint16_t)kb;
            cnt += __popc(bal);
        }
        if (lane == 0) s_count = cnt;
    }
    __syncthreads();
    const int n_tiles = s_count;

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
        const int jt = list[it];
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
    if (n_tiles > 0) issue(0, 0);
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
        const int jt = list[it];
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
        const bool full = jt < qb;       // only the diagonal block needs the causal mask
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float x = s[j][e] * a.scale_log2;
                if (!full) {
                    const int key = j0 + j * 8 + 2 * t4 + (e & 1);
                    const int row = i0 + wr0 + g + 8 * (e >> 1);
                    const bool keep = key <= row;
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

    cp_async_wait<0>();      // (the Q copy, when the block list is empty)
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        l_r[i] += __shfl_xor_sync(0xffffffffu, l_r[i], 1);
        l_r[i] += __shfl_xor_sync(0xffffffffu, l_r[i], 2);
        const int row = i0 + wr0 + g + 8 * i;
        if (row < q_end) {
            // a query that keeps no key at all (its mask row lacks the diagonal block): zero row, flagged
            if (!(l_r[i] > 0.f) && t4 == 0) atomicOr(a.status, FLUX_STATUS_BAD_MASK);
            const float inv = l_r[i] > 0.f ? 1.f / l_r[i] : 0.f;
            __nv_bfloat16 *dst = a.out + ((size_t)(row - a.q_start) * a.Hq + h) * kHeadDim;
#pragma unroll
            for (int nt = 0; nt < 16; ++nt)
                *reinterpret_cast<uint32_t *>(dst + nt * 8 + 2 * t4) =
                    pack_bf16(o[nt][2 * i] * inv, o[nt][2 * i + 1] * inv);
        }
    }
}

}  // namespace

int prefill_blocks_setup()
{
    return check_cuda(cudaFuncSetAttribute(prefill_blocks_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kSmemBytes),
                      "cudaFuncSetAttribute(prefill_blocks_kernel)");
}

int launch_prefill_blocks_mma(flux_plan *p, const void *q, const void *k, const void *v, int q_start, int Nq,
                          const uint8_t *block_mask, int n_kv_blocks, void *out, cudaStream_t st)
{
    const flux_config &c = p->cfg;
    if (n_kv_blocks > kMaxKvBlocks)
        return fail(FLUX_E_CAPACITY, "block mask rows of %d blocks exceed the limit of %d", n_kv_blocks, kMaxKvBlocks);
    BlkArgs a;
    a.q = (const __nv_bfloat16 *)q;
    a.k = (const unsigned char *)k;
    a.v = (const unsigned char *)v;
    a.out = (__nv_bfloat16 *)out;
    a.bm = block_mask;
    a.n_kb = n_kv_blocks;
    a.Hq = c.n_q_heads; a.Hkv = c.n_kv_heads; a.G = p->G; a.q_start = q_start; a.Nq = Nq;
    a.scale_log2 = p->scale_log2;
    a.status = (uint32_t *)((char *)p->ws + p->lay.status);
    dim3 grid((Nq + BM - 1) / BM, c.n_q_heads);
    const int rec = prof_begin(p, FLUX_KERNEL_PREFILL, st);
    prefill_blocks_kernel<<<grid, kWarps * 32, kSmemBytes, st>>>(a);
    prof_end(p, rec, st);
    p->launches++;
    return check_cuda(cudaGetLastError(), "block-mask prefill kernel launch");
}

}  // namespace flux
