// Internal declarations shared by the translation units of libflux_attn.so.
// Nothing here is part of the public ABI (see include/flux_attn.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "flux_attn.h"

namespace flux {

constexpr int kHeadDim = 128;
constexpr int kRowBytes = kHeadDim * 2;  // one head of one token, bf16

// ---- decode kernel geometry -------------------------------------------------
constexpr int kDecWarps = 8;        // warps per CTA, each an independent streaming pipeline
constexpr int kDecTile = 16;        // tokens per pipeline stage of one warp
constexpr int kDecStages = 3;       // cp.async stages per warp
constexpr int kDecStageBytes = kDecTile * kRowBytes * 2;  // K tile + V tile
constexpr int kDecMaxCtas = 512;    // upper bound used to size the workspace
constexpr int kMaxPeers = 8;        // GPUs a decode step's keys can be spread over (one NVSwitch domain)
constexpr int kMaxBatch = 1024;     // prefix tables live in shared memory
constexpr int kDecFusedMaxBatch = 32;   // largest batch the single-launch decode kernel takes
constexpr int kDecFusedAutoBatch = 32;  // largest batch it is chosen for by default
constexpr int kDecFusedMaxKvHeads = 64;
constexpr int kRouterMaxWidth = 4096;   // largest hidden width of the router MLPs (sizes the scratch)

// ---- workspace layout (byte offsets from the workspace base) ----------------
struct WorkspaceLayout {
    size_t status;       // uint32 status word (+ padding)
    size_t debug;        // int32 [max_batch][8] dispatch records
    size_t sched;        // int32 [max_batch + 4] decode schedule table (prefix, span)
    size_t stage_mask;   // uint8 [max_batch][L]
    size_t stage_logits; // fp32  [max_batch][L][2]
    size_t part_o;       // fp32  [slots][G][D]
    size_t part_ml;      // fp32  [slots][G][2]
    size_t host_q;       // bf16  [max_batch][Hq][D]   staging for *_host calls
    size_t host_k;       // bf16  [max_batch][Hkv][D]
    size_t host_v;       // bf16  [max_batch][Hkv][D]
    size_t host_o;       // bf16  [max_batch][Hq][D]
    size_t router;       // fp32 [2*Hq*D] pooled descriptor, then uint64 [3][kRouterMaxWidth] hidden activations (value | launch number << 32)
    size_t router_sync;  // uint32 [8]: barrier counter and exit ticket of the router front end (zero between launches), its launch number
    size_t push_ticket;  // uint32 [8]: CTAs of a pushing merge launch that have stored their rows (zero between launches)
    size_t tickets;      // uint32 [2][kDecFusedMaxBatch][Hkv] arrival / helper counters of the single-launch decode (zero between launches)
    size_t total;
    int64_t slots;
};

WorkspaceLayout workspace_layout(const flux_config &cfg);

// heads of one KV-head group a decode CTA serves at once, and token slices per CTA tile
inline int dec_heads_per_cta(int Hkv) { return Hkv < kDecWarps ? Hkv : kDecWarps; }
inline int dec_slices(int Hkv) { return kDecWarps / dec_heads_per_cta(Hkv); }
inline int dec_head_groups(int Hkv)
{
    int hpc = dec_heads_per_cta(Hkv);
    return (Hkv + hpc - 1) / hpc;
}

struct Dev {
    int n_sms;
    int smem_optin;
    int cc_major;
};

}  // namespace flux

struct flux_plan {
    flux_config cfg;
    flux::Dev dev;
    int G;
    float scale;        // softmax scale
    float scale_log2;   // scale * log2(e)
    void *ws;
    size_t ws_bytes;
    flux::WorkspaceLayout lay;
    const uint8_t *d_mask;  // cached routing decision [mask_B][L], device
    int32_t mask_B;
    int64_t launches;
    int32_t debug_records;  // records the latest call wrote
    uint32_t *touch;        // optional device bitmap of the KV rows read (flux_debug_touched), NULL = off
    int32_t touch_words;    // 32-bit words per request
    int dec_ctas;
    int decode_kernel;      // FLUX_DECODE_*
    int launch_overlap;     // flux_plan_set_launch_overlap
    // optional per-kernel timing (host-side event pool)
    cudaEvent_t *prof_ev;     // 2 * prof_cap events
    int8_t *prof_kind;
    int32_t prof_cap, prof_n;
};

namespace flux {

// error bookkeeping (flux_api.cu)
int fail(int code, const char *fmt, ...);
int check_cuda(cudaError_t e, const char *what);

// kernel launchers; each returns FLUX_OK or a negative code and bumps plan->launches
int launch_router(flux_plan *p, const float *d_logits, const uint8_t *d_mask_in, int B,
                  uint8_t *d_mask_out, cudaStream_t st);
// Layer Router front end: pooled x_Q segments -> encoder -> head -> two logits at d_logits_out
int launch_router_frontend(flux_plan *p, const flux_router_weights *w, const void *q_first, int n_first,
                           const void *q_last, int n_last, float *d_logits_out, cudaStream_t st);
int launch_kv_append(flux_plan *p, int layer, int B, const void *k_new, const void *v_new,
                     void *const *k_caches, void *const *v_caches, const int32_t *pos,
                     cudaStream_t st);
int launch_kv_retain(flux_plan *p, int layer, int req, const void *k_src, const void *v_src,
                     int n, void *k_cache, void *v_cache, cudaStream_t st);
// k_new / v_new non-NULL: the launch also appends the newest token (flux_attn_decode_step);
// head_mask non-NULL: per-KV-head modes [B][Hkv] instead of the routed layer mask (flux_attn_decode_heads)
// part non-NULL: evaluate only the keys [key_begin[b], key_end[b]) and write the merged (O, m, l) of every
// (request, query head) to out_o / out_ml instead of the bf16 output (flux_attn_decode_partial)
struct DecPush {              // where a pushed piece goes (flux_attn_decode_partial_push); world == 0: nowhere
    int world, rank;
    uint32_t seq;
    float *o[kMaxPeers], *ml[kMaxPeers];
    uint32_t *flags[kMaxPeers];
};
struct DecPartial {
    const int32_t *key_begin, *key_end;
    float *out_o, *out_ml;
    DecPush push;
};
int launch_decode(flux_plan *p, int layer, int B, const void *q, const void *const *k_caches,
                  const void *const *v_caches, const int32_t *ctx_len, void *out,
                  cudaStream_t st, const void *k_new = nullptr, const void *v_new = nullptr,
                  const uint8_t *head_mask = nullptr, const DecPartial *part = nullptr);
int launch_combine_sets(flux_plan *p, const float *po, const float *pml, int n_sets, int n_rows, void *out, cudaStream_t st,
                        const uint32_t *flags = nullptr, uint32_t seq = 0, long long wait_cycles = 0);
int launch_prefill(flux_plan *p, int layer, int req, const void *q, const void *k, const void *v,
                   int q_start, int Nq, void *out, cudaStream_t st);
// bracket a dominant-kernel launch with events when profiling is on
int prof_begin(flux_plan *p, int kind, cudaStream_t st);   // returns record index or -1
void prof_end(flux_plan *p, int rec, cudaStream_t st);
int launch_prefill_blocks(flux_plan *p, const void *q, const void *k, const void *v, int q_start, int Nq,
                          const uint8_t *block_mask, int n_kv_blocks, void *out, cudaStream_t st);
int launch_wait_probe(flux_plan *p, long long limit_cycles, cudaStream_t st);
int decode_setup(flux_plan *p);   // one-time attribute setting for the decode kernels
int decode_fused_setup(flux_plan *p);
int prefill_setup(flux_plan *p);
int router_setup(flux_plan *p);

}  // namespace flux
