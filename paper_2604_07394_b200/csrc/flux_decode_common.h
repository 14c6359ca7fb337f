// Pieces shared by the two decode kernels: launch arguments, the per-request row ranges of
// Eq. 1 / Eq. 2, and the flash-attention update of one warp over one 16-key tile.
#pragma once

#include <math.h>

#include "flux_internal.h"
#include "flux_mma_util.h"

namespace flux {

constexpr float kNegBig = -1.0e30f;  // finite stand-in for "no key seen yet"

struct DecArgs {
    const __nv_bfloat16 *q;
    const void *const *k_caches;
    const void *const *v_caches;
    const int32_t *ctx_len;
    const uint8_t *mask;
    int B, L, layer, Hq, Hkv, G, S, W, layout, max_context;
    float scale_log2;
    float *part_o;
    float *part_ml;
    int32_t *debug;
    int32_t *sched;
    uint32_t *status;
    __nv_bfloat16 *out;
    // fused append (flux_attn_decode_step): the newest token's K, V rows [B][Hkv][D]; NULL otherwise
    const unsigned char *k_new;
    const unsigned char *v_new;
    uint32_t *touch;            // debug bitmap of the cache rows read ([B][touch_words]), or NULL
    int touch_words;
    // head-level comparison mode (flux_attn_decode_heads): uint8 [B][Hkv], 1 = the KV head's group
    // attends densely, 0 = sink + window; NULL in the routed (layer-level) calls
    const uint8_t *head_mask;
    // single-launch kernel: per (request, KV head) the count of CTAs that have announced their partials, and the
    // count of CTAs that have started merging them; both zero between launches
    uint32_t *tickets;
    uint32_t *done;
    // single-launch kernel only: schedule and first tile loads before the grid-dependency wait
    int overlap;
    // partial evaluation over a key range (flux_attn_decode_partial): positions [key_begin[b], key_end[b]) of each
    // request, and where the merged (O, m, l) of every (request, query head) goes instead of the bf16 output
    const int32_t *key_begin, *key_end;
    float *pout_o, *pout_ml;
    // pushed pieces (flux_attn_decode_partial_push): the merged piece of every (request, query head) goes into slot
    // push_rank of each of push_world gather buffers (this GPU's own and its peers', all addresses valid here), then
    // entry push_rank of each one's flag array is set to push_seq.  push_world == 0: off.
    int push_world, push_rank;
    uint32_t push_seq;
    float *push_o[kMaxPeers], *push_ml[kMaxPeers];
    uint32_t *push_flags[kMaxPeers];
    uint32_t *push_ticket;      // workspace counter: CTAs of the merge launch that have stored their rows (zero between launches)
};

// What one request contributes to this layer's launch.
struct ReqInfo {
    int n;       // context length after clamping
    int mode;    // 1 FA, 0 SA
    int n_eff;   // rows the kernel reads
    int split;   // virtual rows >= split are shifted by `shift` (window part of a FULL cache)
    int shift;
};

__device__ __forceinline__ ReqInfo req_info(int n_raw, int mode_raw, int S, int W, int layout,
                                            int max_context, uint32_t *status)
{
    ReqInfo r;
    int n = n_raw;
    if (n > max_context) {
        atomicOr(status, FLUX_STATUS_BAD_LENGTH);
        n = max_context;
    }
    if (n < 0) n = 0;
    if (mode_raw > 1) atomicOr(status, FLUX_STATUS_BAD_MASK);
    r.n = n;
    r.mode = mode_raw != 0 ? 1 : 0;
    r.split = 0x7fffffff;
    r.shift = 0;
    if (r.mode == 1 || n <= S + W) {
        r.n_eff = n;  // SA with sink + window >= n keeps every row
    } else {
        r.n_eff = S + W;
        if (layout == FLUX_KV_FULL) {  // rows [0,S) then rows [n-W, n)
            r.split = S;
            r.shift = n - W - S;
        }  // COMPACT_SA: the S + W slots are exactly the kept rows, in slot order
    }
    return r;
}

// Restricts a request to the key positions [kb, ke).  A request that walks its rows densely (FA, or SA while sink +
// window still cover the context) reads rows kb .. ke - 1; a sparse request is taken whole by the range that holds
// its newest position and skipped by every other range (its kept rows are few: splitting them gains nothing).
__device__ __forceinline__ void dec_restrict(ReqInfo &r, int kb, int ke, int S, int W)
{
    kb = kb < 0 ? 0 : kb;
    ke = ke > r.n ? r.n : ke;
    if (r.mode == 1 || r.n <= S + W) {
        r.split = 0;
        r.shift = kb;
        r.n_eff = ke > kb ? ke - kb : 0;
    } else if (!(kb <= r.n - 1 && r.n - 1 < ke)) {
        r.n_eff = 0;
    }
}

// Cache row of the token a fused-append launch stores for a request (-1: nothing to store).
__device__ __forceinline__ int dec_new_row(const ReqInfo &r, bool appending, int S, int W, int layout)
{
    const bool compact = layout == FLUX_KV_COMPACT_SA && r.mode == 0;
    const int pnew = r.n - 1;   // the newest token sits at position n - 1; in a compact sparse cache that is a ring slot
    if (!appending || pnew < 0) return -1;
    return (compact && pnew >= S) ? S + (pnew - S) % W : pnew;
}

// Dispatch record of one request: mode, layer, request, length, and the two cache-row ranges read.
__device__ __forceinline__ void dec_write_record(int32_t *d, const ReqInfo &r, int layer, int b)
{
    d[0] = r.mode; d[1] = layer; d[2] = b; d[3] = r.n;
    d[4] = 0;
    d[5] = (r.split < r.n_eff) ? r.split : r.n_eff;
    d[6] = (r.split < r.n_eff) ? r.split + r.shift : 0;
    d[7] = (r.split < r.n_eff) ? r.n_eff + r.shift : 0;
}

// Query rows of one KV head's group as A fragments of m16n8k16 (rows >= G are zero).
__device__ __forceinline__ void dec_load_q(uint32_t (&qf)[8][4], const __nv_bfloat16 *qb, int G, int lane)
{
    const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int row = g + 8 * (e & 1);
            const int col = kk * 16 + 2 * t4 + 8 * (e >> 1);
            qf[kk][e] = row < G ? *reinterpret_cast<const uint32_t *>(qb + (size_t)row * kHeadDim + col) : 0u;
        }
    }
}

__device__ __forceinline__ void dec_state_reset(float (&o)[16][4], float (&m_r)[2], float (&l_r)[2])
{
#pragma unroll
    for (int nt = 0; nt < 16; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[nt][e] = 0.f;
    m_r[0] = m_r[1] = kNegBig;
    l_r[0] = l_r[1] = 0.f;
}

// One warp, one tile of kDecTile keys staged in shared memory (K at kb, V at vb, 256-byte rows with
// the 16-byte chunks XOR-swizzled by the row): S = Q K^T, online softmax in the log2 domain, O += P V.
// Keys at or beyond n_valid are masked out.
__device__ __forceinline__ void dec_attend_tile(float (&o)[16][4], float (&m_r)[2], float (&l_r)[2],
                                                const uint32_t (&qf)[8][4], uint32_t kb, uint32_t vb,
                                                int n_valid, float scale_log2, int lane)
{
    const int t4 = lane & 3;
    float s[2][4];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) s[j][e] = 0.f;
    {
        const int mi = lane >> 3, rr = lane & 7;
        const int key = (mi >> 1) * 8 + rr;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            const int chunk = kk * 2 + (mi & 1);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(b0, b1, b2, b3, kb + key * kRowBytes + ((chunk ^ rr) << 4));
            mma_bf16(s[0], qf[kk], b0, b1);
            mma_bf16(s[1], qf[kk], b2, b3);
        }
    }
    // scale into the log2 domain, mask the ragged tail
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int key = j * 8 + 2 * t4 + (e & 1);
            s[j][e] = key < n_valid ? s[j][e] * scale_log2 : -INFINITY;
        }
    // online softmax for rows g and g + 8
    float alpha[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        float mx = fmaxf(fmaxf(s[0][2 * i], s[0][2 * i + 1]), fmaxf(s[1][2 * i], s[1][2 * i + 1]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_r[i], mx);
        alpha[i] = fast_exp2(m_r[i] - m_new);
        m_r[i] = m_new;
        float rs = 0.f;
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const float p = fast_exp2(s[j][2 * i + e] - m_new);
                s[j][2 * i + e] = p;
                rs += p;
            }
        l_r[i] = l_r[i] * alpha[i] + rs;
    }
    uint32_t pa[4];
    pa[0] = pack_bf16(s[0][0], s[0][1]);
    pa[1] = pack_bf16(s[0][2], s[0][3]);
    pa[2] = pack_bf16(s[1][0], s[1][1]);
    pa[3] = pack_bf16(s[1][2], s[1][3]);
    // O = alpha * O + P V
    {
        const int mi = lane >> 3, rr = lane & 7;
        const int key = (mi & 1) * 8 + rr;
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) {
            const int chunk = dt * 2 + (mi >> 1);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4_trans(b0, b1, b2, b3, vb + key * kRowBytes + ((chunk ^ rr) << 4));
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
                float(&acc)[4] = o[2 * dt + h2];
                acc[0] *= alpha[0];
                acc[1] *= alpha[0];
                acc[2] *= alpha[1];
                acc[3] *= alpha[1];
            }
            mma_bf16(o[2 * dt], pa, b0, b1);
            mma_bf16(o[2 * dt + 1], pa, b2, b3);
        }
    }
}

}  // namespace flux
