/*
 * flux_attn.h -- C ABI of libflux_attn.so: routed hybrid attention for one B200.
 *
 * The library runs the per-layer hot path of Flux Attention: a cached hard
 * routing bit per (request, layer) sends the layer to causal Full Attention
 * (Eq. 1) or to Sparse Attention over a condensed KV subset (Eq. 2; here the
 * streaming subset: an attention sink of `sink` leading positions plus a local
 * window of the `window` latest positions, query included), in prefill and in
 * autoregressive decode.
 *
 * General rules
 *  - Every entry point returns FLUX_OK (0) or a negative FLUX_E_* code; none
 *    throws, exits or prints.  flux_last_error() gives a message for the last
 *    failure on the calling thread.
 *  - The library allocates no device memory.  The caller owns every device
 *    buffer, including the workspace whose size flux_workspace_size() reports;
 *    a plan owns host memory only.
 *  - "device" pointers are CUDA global-memory addresses valid on the current
 *    device; "host" pointers are ordinary CPU addresses.  Each argument says
 *    which it is.  Device buffers must be 16-byte aligned.
 *  - Calls are asynchronous on `stream` (a cudaStream_t passed as void*, NULL
 *    for the default stream) unless stated otherwise.  Conditions that only the
 *    device can see (a mask byte outside {0,1}, a NaN logit, a context length
 *    outside [1, max_context], a wait that ran out) set bits in a device status
 *    word; flux_plan_status() synchronises the stream and returns them.
 *  - All tensors are bfloat16 unless stated otherwise; accumulation is fp32.
 *  - Layouts: Q and O rows are [n_q_heads][head_dim]; a KV cache of one
 *    (layer, request) is [rows][n_kv_heads][head_dim], token-major, so one
 *    token's keys of all heads are one contiguous 2*n_kv_heads*head_dim-byte row.
 *    Query head h reads KV head h / (n_q_heads / n_kv_heads).
 *  - Mask encoding (Sec. 3.1, "Deterministic Inference via Hard Routing"):
 *    1 = FA, 0 = SA.
 */
#ifndef FLUX_ATTN_H
#define FLUX_ATTN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FLUX_OK                   0
#define FLUX_E_INVALID_ARG       -1  /* null / misaligned pointer, bad index, bad size          */
#define FLUX_E_UNSUPPORTED_SHAPE -2  /* head_dim != 128, n_q_heads % n_kv_heads != 0, G > 16    */
#define FLUX_E_CAPACITY          -3  /* batch or length beyond what the plan was created for    */
#define FLUX_E_WORKSPACE         -4  /* workspace missing or too small                          */
#define FLUX_E_DEVICE_TIMEOUT    -5  /* a bounded device-side wait gave up                      */
#define FLUX_E_CUDA              -6  /* a CUDA runtime / driver call failed                     */
#define FLUX_E_DEVICE_FLAG       -7  /* device-side input check failed (see status bits)        */

/* bits of the device status word returned by flux_plan_status() */
#define FLUX_STATUS_BAD_MASK      1u   /* mask byte not 0/1                                     */
#define FLUX_STATUS_NAN_LOGIT     2u   /* routing logit is NaN                                  */
#define FLUX_STATUS_BAD_LENGTH    4u   /* ctx_len / pos outside [1, max_context]                */
#define FLUX_STATUS_WAIT_EXPIRED  8u   /* an mbarrier wait hit its iteration limit              */

#define FLUX_KV_FULL        0  /* every layer's cache holds every position: row = position          */
#define FLUX_KV_COMPACT_SA  1  /* an SA layer's cache holds sink + window rows only (Sec. 3.3)      */

typedef struct {
    int32_t n_layers;
    int32_t n_q_heads;
    int32_t n_kv_heads;
    int32_t head_dim;       /* must be 128                                                      */
    int32_t sink;           /* S >= 0: leading positions every SA query keeps                   */
    int32_t window;         /* W >= 1: latest positions an SA query keeps, itself included      */
    float   softmax_scale;  /* 0 selects 1/sqrt(head_dim); Eq. 1 leaves the scale out           */
    int32_t max_batch;      /* largest B any call will pass                                     */
    int32_t max_context;    /* largest context length; every full cache has >= this many rows   */
    int32_t kv_layout;      /* FLUX_KV_FULL or FLUX_KV_COMPACT_SA                               */
} flux_config;

typedef struct flux_plan flux_plan; /* opaque host object */

/* Plan life cycle.  Creating a plan validates the configuration and queries the
 * current device (SM count, shared memory); it launches nothing.  Host memory
 * only; flux_plan_destroy frees it.  *plan is set to NULL on failure. */
int flux_plan_create(const flux_config *cfg, flux_plan **plan);
int flux_plan_destroy(flux_plan *plan);

/* Device workspace (split-K partials, status word, debug records, staging for
 * the *_host calls).  bytes_out (host) receives the size for this configuration.
 * The caller allocates it (256-byte aligned), zero-fills it once, and hands it
 * over; it must stay valid and untouched by others while the plan is in use. */
int flux_workspace_size(const flux_config *cfg, size_t *bytes_out);
int flux_plan_set_workspace(flux_plan *plan, void *workspace /*device*/, size_t bytes);

/* Layer Router front end (Sec. 3.1, "Architecture and Feature Extraction"; Appendix D.1): from
 * the layer's query tensor x_Q to the routing logits of one (request, layer).
 *   f  = concat(mean over tokens of q_first, mean over tokens of q_last)      [2*n_q_heads*head_dim]
 *        (Prefill-Suffix Pooling; index = segment*Hq*D + head*D + channel)
 *   h1 = silu(w_enc1 f + b_enc1);  u = w_enc2 h1 + b_enc2                      Context Encoder
 *   h2 = silu(w_head1 u + b_head1); (pi_FA, pi_SA) = w_head2 h2 + b_head2      Router Head
 * The paper names these stages but not the pooling operator, the widths or the activation; the
 * token mean and silu(x) = x / (1 + exp(-x)) are this library's choice.
 *   q_first, q_last  bf16 [n_first][n_q_heads][head_dim] and [n_last][..][..], device: the first
 *                    and the last prompt tokens of x_Q (the paper pools 100 + 100; shorter
 *                    prompts pass min(100, n) tokens each, the two may overlap).  n_* >= 1.
 *   w                host struct of device pointers: weights bf16 row-major [out][in], biases
 *                    fp32; widths enc_dim (E) and head_hidden (R) multiples of 8, <= 4096;
 *                    w_enc1 [E][2*Hq*D], w_enc2 [E][E], w_head1 [R][E], w_head2 [2][R] (row 0 = FA).
 *   logits_out       fp32 [2] on the device, 8-byte aligned, e.g. the (request, layer) slot of the
 *                    [B][n_layers][2] array later given to flux_router_apply.
 * One launch on `stream` (pooling + four matrix-vector products, fp32 accumulation, a fixed
 * summation order); scratch is in the workspace, so calls for different layers must be
 * stream-ordered.  Cost does not depend on the prompt length.  The launch may begin while the
 * kernel before it in the stream is still draining, and reads the WEIGHTS AND BIASES (nothing
 * else) before that kernel has finished: the work enqueued immediately before this call must not
 * be what writes them.  The kernel's CTAs (one per SM) wait for one another between stages; the
 * waits are bounded (about a second, then FLUX_STATUS_WAIT_EXPIRED in the status word and
 * unspecified logits), which only a kernel of another stream that holds SMs for that long can
 * cause.  Errors: NULL / misaligned pointers, n_* < 1 -> FLUX_E_INVALID_ARG; widths
 * not multiples of 8 -> FLUX_E_UNSUPPORTED_SHAPE; widths > 4096 -> FLUX_E_CAPACITY. */
typedef struct {
    int32_t enc_dim;       /* E */
    int32_t head_hidden;   /* R */
    const void *w_enc1;  const float *b_enc1;
    const void *w_enc2;  const float *b_enc2;
    const void *w_head1; const float *b_head1;
    const void *w_head2; const float *b_head2;
} flux_router_weights;
int flux_router_forward(flux_plan *plan, const flux_router_weights *w, const void *q_first, int32_t n_first,
                        const void *q_last, int32_t n_last, float *logits_out /*device*/, void *stream);

/* Hard routing, once per request batch at prefill; the result is cached for all
 * decode steps (Sec. 3.1 "Deterministic Inference via Hard Routing", Sec. 3.3).
 *   logits       fp32 [B][n_layers][2], FA logit first; device or host memory;
 *                ignored when mask_or_null is given.
 *   mask_or_null uint8 [B][n_layers] ready-made decisions (device or host), or NULL.
 *   mask_out     uint8 [B][n_layers], device; receives 1 where pi_FA >= pi_SA (a tie
 *                keeps FA), else 0.  The plan remembers this pointer: later calls
 *                read the routing decision from it, so it must stay alive.
 * Host inputs are validated on the host (NaN logit or mask byte outside {0,1}
 * -> FLUX_E_INVALID_ARG, nothing launched) and staged through the workspace;
 * device inputs are checked by the kernel (status bits).  B <= max_batch. */
int flux_router_apply(flux_plan *plan, const float *logits, const uint8_t *mask_or_null,
                      int32_t B, uint8_t *mask_out, void *stream);

/* Prefill of one layer for one request (Eq. 1 or Eq. 2 by mask[req][layer]),
 * causal.  Query rows sit at absolute positions q_start .. q_start+Nq-1 (chunked
 * prefill, Appendix D.3 "chunk size"); k, v hold positions 0 .. q_start+Nq-1 as
 * [rows][n_kv_heads][head_dim] with row = position (a FULL-layout cache or the
 * projection output itself).
 *   q, out   [Nq][n_q_heads][head_dim], device.    k, v  device, read only.
 * Nq == 0 is a successful no-op.  q_start + Nq <= max_context. */
int flux_attn_prefill(flux_plan *plan, int32_t layer, int32_t req, const void *q,
                      const void *k, const void *v, int32_t q_start, int32_t Nq,
                      void *out, void *stream);

/* Prefill of one request under a block mask: Sparse Attention (Eq. 2) whose condensed key subset
 * is given in blocks of 64 positions, the unit in which the sparse kernels the paper runs select
 * keys (Appendix D.3, "block size"; Sec. 4.1 names the block patterns).  Query position i attends
 * to { j <= i : block_mask[i / 64][j / 64] != 0 }: causality still holds inside a kept block.
 *   block_mask  uint8 [n_q_blocks][n_kv_blocks], device, row-major; rows are ABSOLUTE query blocks
 *               (row (q_start + r) / 64 serves chunk row r), so one matrix serves every chunk;
 *               entries beyond the diagonal are ignored.  n_kv_blocks <= 4096 (else FLUX_E_CAPACITY).
 *   q, out      [Nq][n_q_heads][head_dim], device; k, v as in flux_attn_prefill.
 *   q_start     multiple of 64.
 * Independent of the routing decision (no layer / request arguments).  A query whose mask row
 * keeps no block up to its own gets a zero output row and raises FLUX_STATUS_BAD_MASK. */
int flux_attn_prefill_blocks(flux_plan *plan, const void *q, const void *k, const void *v,
                             int32_t q_start, int32_t Nq, const uint8_t *block_mask,
                             int32_t n_kv_blocks, void *out, void *stream);

/* Sparse-decode KV retention after prefill (Sec. 3.3: a sparse layer keeps only
 * the rows its kernel needs).  Copies, for one (layer, request), the rows of
 * k_src/v_src ([n][n_kv_heads][head_dim], row = position) that decode will need
 * into the layer's cache: all n rows for an FA layer or the FULL layout; for an
 * SA layer in the COMPACT_SA layout rows [0,S) to slots [0,S) and rows
 * [max(S,n-W), n) to slot S + ((position - S) mod W).  All pointers device. */
int flux_kv_retain(flux_plan *plan, int32_t layer, int32_t req, const void *k_src,
                   const void *v_src, int32_t n, void *k_cache, void *v_cache, void *stream);

/* Append one new token per request to the caches of one layer (Sec. 3.3).
 *   k_new, v_new       [B][n_kv_heads][head_dim], device.
 *   k_caches, v_caches device arrays of B device pointers (this layer's cache of
 *                      each request).
 *   pos                int32 [B], device: position being written (= context length
 *                      before the append).  pos < 0 skips the request.
 * FA layers and the FULL layout write row pos; SA layers in COMPACT_SA write
 * slot pos (pos < S) or S + ((pos - S) mod W). */
int flux_kv_append(flux_plan *plan, int32_t layer, int32_t B, const void *k_new,
                   const void *v_new, void *const *k_caches, void *const *v_caches,
                   const int32_t *pos, void *stream);

/* One decode step of one layer for the whole batch: one query row per request at
 * position ctx_len-1 (its K, V already appended).  FA requests stream the whole
 * cache, SA requests only their sink + window rows (Appendix C.3); one launch serves
 * mixed modes, split over all SMs in equal-byte spans, followed by a combine pass (small
 * batches: one launch does both, see flux_debug_decode_kernel).
 *   q, out    [B][n_q_heads][head_dim], device.
 *   k_caches, v_caches  device arrays of B device pointers.
 *   ctx_len   int32 [B], device: context length including the new token;
 *             <= 0 marks an inactive request (its output row is zero-filled). */
int flux_attn_decode(flux_plan *plan, int32_t layer, int32_t B, const void *q,
                     const void *const *k_caches, const void *const *v_caches,
                     const int32_t *ctx_len, void *out, void *stream);

/* flux_kv_append and flux_attn_decode of one layer in one launch (Sec. 3.3: the new token's K, V
 * join the cache, then the token attends): the kernel stores k_new / v_new at position
 * ctx_len - 1 of each request's cache (ring slot for a compact sparse cache) and reads that one
 * row from k_new / v_new instead of the cache, so no second kernel and no ordering between the
 * two is needed.  Same results as the two calls with pos = ctx_len - 1.  At small batches the
 * saved launch is a visible part of a decode step.
 *   k_new, v_new  [B][n_kv_heads][head_dim], device.   Everything else as in flux_attn_decode;
 *   requests with ctx_len <= 0 are skipped (nothing stored, zero output row). */
int flux_attn_decode_step(flux_plan *plan, int32_t layer, int32_t B, const void *q,
                          const void *k_new, const void *v_new, void *const *k_caches,
                          void *const *v_caches, const int32_t *ctx_len, void *out, void *stream);

/* Head-level sparsity, the alternative the paper argues against (Sec. 2.3 "Motivational
 * Observations", Fig. 1(b); Appendix C.3 "Implementation of Sparsity Baselines"): inside ONE layer
 * some KV heads (with their query-head groups) attend densely and the others keep only sink +
 * window.  Same arithmetic as flux_attn_decode, but the mode comes per (request, KV head) from
 * head_mask instead of the cached layer mask, so the routed stack and a head-level stack of the
 * same KV byte budget can be timed on the same kernel.  The request is walked over its whole
 * length if any of its heads is dense; warps that own a sparse head read only its sink + window
 * rows and idle for the rest of the walk, and the dense heads' rows are 256-byte pieces of the
 * token-major cache rows -- the fragmented access and the intra-layer imbalance the paper describes.
 *   head_mask  uint8 [B][n_kv_heads] on the device: 1 = dense (Eq. 1), 0 = sink + window (Eq. 2);
 *              other values set FLUX_STATUS_BAD_MASK and count as dense.
 *   other arguments as flux_attn_decode; caches must be in the FLUX_KV_FULL layout
 *   (else FLUX_E_UNSUPPORTED_SHAPE).  No routing call is needed beforehand. */
int flux_attn_decode_heads(flux_plan *plan, int32_t B, const void *q, const void *const *k_caches,
                           const void *const *v_caches, const int32_t *ctx_len,
                           const uint8_t *head_mask /*device*/, void *out, void *stream);

/* Decode step for callers that cannot allocate device memory at all.  (The paper
 * has no counterpart: this is a packaging variant of flux_attn_decode, not part of
 * the method.)  Who needs it: code that runs inside a host program which owns all
 * device memory and passes in only the operator's own tensors, and loops that may
 * not risk the device-wide synchronisation an allocation can cause.  The split-K
 * scratch that flux_attn_decode keeps in the caller's workspace sits here in a
 * fixed array of about 9.6 MB inside the library image, held on every GPU the
 * process uses until it exits.  No plan and no workspace are needed; the call
 * makes no cudaMalloc / cudaFree and uses no allocating library routine.
 *   cfg        shapes as for flux_plan_create (max_batch is ignored).
 *   mask       uint8 [B][n_layers], device: the routing decision (1 FA, 0 SA).
 *   q, out, k_caches, v_caches, ctx_len: as in flux_attn_decode, all device.
 *   status_out optional device uint32: receives the FLUX_STATUS_* bits of this call.
 * Limits (beyond them the call returns FLUX_E_CAPACITY and launches nothing):
 * B <= 64, n_q_heads / n_kv_heads <= 8, n_kv_heads <= 16.
 * The first call on each device resolves the array's device address and sets a
 * kernel attribute; make that first call before any stream capture begins.
 * All calls on a device share the one array, which keeps the previous call's
 * contents (the status word is cleared at the start of each call): calls whose
 * kernels may overlap on the GPU -- different streams, or several host threads --
 * race on it and must be serialised by the caller. */
int flux_attn_decode_noalloc(const flux_config *cfg, int32_t layer, int32_t B,
                             const uint8_t *mask, const void *q,
                             const void *const *k_caches, const void *const *v_caches,
                             const int32_t *ctx_len, void *out, uint32_t *status_out,
                             void *stream);

/* The same decode step for callers whose activations live in host memory: brings
 * q, k_new, v_new (host) to the device, appends, attends, and delivers the result
 * to out (host).  With pinned (page-locked) buffers the kernels read the inputs from
 * host memory and write the result there directly, each byte crossing the bus once
 * and no copy operation in the stream (three launches); with pageable buffers the
 * call stages them through the workspace with four asynchronous copies.
 * Asynchronous on `stream` like the rest; the host buffers must stay untouched
 * until the stream is synchronised.  The caches, pointer tables, pos and ctx_len
 * stay on the device. */
int flux_attn_decode_host(flux_plan *plan, int32_t layer, int32_t B, const void *q_host,
                          const void *k_new_host, const void *v_new_host,
                          void *const *k_caches, void *const *v_caches, const int32_t *pos,
                          const int32_t *ctx_len, void *out_host, void *stream);

/* Prefill for host-resident activations: q (host) is copied to the device buffer
 * q_dev, the layer runs as flux_attn_prefill, and out_dev is copied to out_host. */
int flux_attn_prefill_host(flux_plan *plan, int32_t layer, int32_t req, const void *q_host,
                           void *q_dev, const void *k, const void *v, int32_t q_start,
                           int32_t Nq, void *out_dev, void *out_host, void *stream);

/* Synchronises `stream`, reads the device status word and clears it.  Returns
 * FLUX_OK with *status_bits == 0, FLUX_E_DEVICE_TIMEOUT if a wait expired, or
 * FLUX_E_DEVICE_FLAG for the input-check bits.  status_bits (host) may be NULL.
 * A kernel that gave up on a wait leaves its hand-over state in the workspace wherever it
 * stood; when the word reports a timeout this call also puts that state (the arrival counters
 * of the single-launch decode, the router front end's counters, launch number and tagged
 * activations) back to zero on `stream`, so the calls that follow start clean. */
int flux_plan_status(flux_plan *plan, uint32_t *status_bits, void *stream);

/* Dispatch record of the latest flux_attn_decode / flux_attn_prefill on this
 * plan, for verification: synchronises `stream` and copies n_records records of
 * 8 int32 each to records_out (host):
 *   { mode (1 FA, 0 SA), layer, request, n, a_begin, a_end, b_begin, b_end }
 * where [a_begin,a_end) and [b_begin,b_end) are the cache rows the kernel reads
 * for the newest query row (b is empty for FA).  Decode writes one record per
 * request, prefill one record.  n_records_out (host) receives the count. */
int flux_debug_dispatch(flux_plan *plan, int32_t *records_out, int32_t max_records,
                        int32_t *n_records_out, void *stream);

/* Which KV rows the kernels actually read, for verification.  While a bitmap is set, the decode
 * kernel sets bit r of request b's words for every cache row r (slot, in a compact sparse cache)
 * whose K and V it loads, and the tcgen05 prefill kernel sets the bits of every position of every
 * KV tile it loads (request words 0; tiles are 128 positions, clipped to the rows present).
 *   bitmap  uint32 [max_batch][words_per_request], device, zeroed by the caller; NULL turns the
 *           recording off (the default).  words_per_request * 32 >= max_context.
 * The bits accumulate over launches until the caller clears the buffer. */
int flux_debug_touched(flux_plan *plan, uint32_t *bitmap, int32_t words_per_request);

/* Per-kernel device timing for roofline reports.  flux_profile_enable creates
 * max_records pairs of CUDA events (host objects; max_records == 0 turns
 * profiling off and destroys them); while enabled, every launch of a dominant
 * kernel (FLUX_KERNEL_DECODE: the split-K decode kernel, FLUX_KERNEL_PREFILL: the
 * prefill attention kernel) is bracketed by two event records on its stream until
 * the pairs run out.  flux_profile_read synchronises `stream`, sums the elapsed
 * time of the recorded launches of `kind` into *total_ms, stores their count in
 * *launches (both host), and resets the recorder. */
#define FLUX_KERNEL_DECODE  0
#define FLUX_KERNEL_PREFILL 1
int flux_profile_enable(flux_plan *plan, int32_t max_records);
int flux_profile_read(flux_plan *plan, int32_t kind, double *total_ms, int64_t *launches,
                      void *stream);

/* A decode step evaluated in pieces over disjoint key ranges, and the merge of the pieces: the building blocks for
 * spreading one long context over several GPUs (each holds a range of the cache rows, evaluates its piece, the
 * pieces are exchanged -- B * n_q_heads * 130 floats per piece -- and merged).  Eq. 1 / Eq. 2 are sums over keys,
 * so pieces over disjoint key sets merge exactly, by rescaling with the difference of their maxima.
 *
 * flux_attn_decode_partial: as flux_attn_decode, restricted per request to the key positions
 * [key_begin[b], key_end[b]) (device int32 arrays; clamped to [0, ctx_len[b]]).  A request that reads its rows
 * densely (FA, or SA while sink + window still cover the context) reads exactly those rows; a sparse request is
 * evaluated whole by the call whose range holds its newest position ctx_len[b] - 1 and yields an empty piece in
 * every other call.  Instead of an output row the call writes, for every (request, query head), the piece
 *   part_o  fp32 [B][n_q_heads][head_dim]  sum over the range's kept keys of 2^(s_j - m) V_j   (not normalised)
 *   part_ml fp32 [B][n_q_heads][2]         m = the maximum scaled score in log2 units (s_j = scale * log2(e) * q.k_j;
 *                                          -1e30 for an empty piece), l = sum of 2^(s_j - m)
 * both device memory.  Always runs the two-launch kernels.
 *
 * flux_attn_combine: merges n_sets pieces laid out [n_sets][B][n_q_heads][...] (what an all-gather of the ranks'
 * pieces produces) into out bf16 [B][n_q_heads][head_dim]: m = max m_s, O = sum_s O_s 2^(m_s - m), l likewise,
 * out = O / l (a row whose pieces are all empty is zero).
 *
 * The exchange without a library call (the paper has no counterpart: it runs on one GPU).  Every rank owns a gather
 * buffer gather_o fp32 [world][B][n_q_heads][head_dim], gather_ml fp32 [world][B][n_q_heads][2] and a flag array
 * uint32 [world], zero-filled once, and knows the addresses of all ranks' three arrays as they are mapped on ITS
 * GPU (its own plainly, the peers' through peer access / IPC or symmetric memory; on one NVSwitch domain: up to 8).
 * flux_attn_decode_partial_push evaluates this rank's piece like flux_attn_decode_partial and its merge kernel
 * stores every row straight into slot `rank` of every rank's gather buffer (plain stores to peer memory), then --
 * after a system-scope fence by every CTA and a ticket among them -- sets entry `rank` of every rank's flag array to
 * `seq` (release, system scope).  flux_attn_combine_wait is flux_attn_combine over this rank's own gather buffer,
 * each CTA first waiting (acquire, system scope) until all `world` flags equal `seq`.  The wait is bounded:
 * wait_cycles SM clock cycles (0 = about a second), then FLUX_STATUS_WAIT_EXPIRED and `out` is left unwritten.
 * `seq` is any non-zero value that differs from the one used for the previous exchange through the same buffers
 * (a step counter).  A rank may push exchange k + 1 into a buffer only when every rank has finished merging exchange
 * k out of it: use one buffer set per layer (a rank cannot finish layer l + 1 of a step before every rank has
 * merged layer l of it), or two sets alternately.  Both kernels of the pushing call and the waiting merge never wait
 * for a kernel of the same GPU: the writers of the flags are kernels on other GPUs.  Errors: as the calls above;
 * world outside [1, 8], rank outside [0, world), seq == 0 -> FLUX_E_INVALID_ARG. */
typedef struct {
    int32_t world, rank;
    float *gather_o[8];      /* rank p's gather_o as addressable from this GPU */
    float *gather_ml[8];
    uint32_t *flags[8];
} flux_peer_set;
int flux_attn_decode_partial_push(flux_plan *plan, int32_t layer, int32_t B, const void *q, const void *const *k_caches,
                                  const void *const *v_caches, const int32_t *ctx_len, const int32_t *key_begin /*device*/,
                                  const int32_t *key_end /*device*/, const flux_peer_set *peers /*host*/, uint32_t seq,
                                  void *stream);
int flux_attn_combine_wait(flux_plan *plan, int32_t B, int32_t world, const float *gather_o, const float *gather_ml,
                           const uint32_t *flags /*device, this rank's own*/, uint32_t seq, int64_t wait_cycles,
                           void *out /*device bf16 [B][n_q_heads][head_dim]*/, void *stream);
int flux_attn_decode_partial(flux_plan *plan, int32_t layer, int32_t B, const void *q, const void *const *k_caches,
                             const void *const *v_caches, const int32_t *ctx_len, const int32_t *key_begin,
                             const int32_t *key_end, float *part_o, float *part_ml, void *stream);
int flux_attn_combine(flux_plan *plan, int32_t B, int32_t n_sets, const float *part_o, const float *part_ml, void *out,
                      void *stream);

/* Launch overlap for the single-launch decode kernel (off by default).  With it on, a decode launch
 * builds its schedule and requests its first K / V tiles while the previous kernel in the stream is
 * still draining, and waits for that kernel only before it reads the query rows, the newest K / V row
 * (position ctx_len - 1, from the cache or from k_new / v_new) and before it writes anything.  The
 * caller promises in return that the kernel enqueued immediately before each decode call on the same
 * stream does not write: ctx_len, the routing mask, the pointer tables, or cache rows of the layer
 * being read at positions below ctx_len - 1.  (A decode call of the previous layer, flux_kv_append and
 * flux_attn_decode_step of any layer, and kernels that only produce q / k_new / v_new all qualify.)
 * Results are the same either way; the two-launch kernels ignore the setting. */
int flux_plan_set_launch_overlap(flux_plan *plan, int32_t on);

/* Which kernels flux_attn_decode / flux_attn_decode_step launch.  FLUX_DECODE_AUTO (the default)
 * runs the single-launch kernel for batches of at most 32 requests and at most 64 KV heads (one launch
 * does the split-K attention and the merge: the first CTAs of a (request, KV head) merge one query head
 * each once all its CTAs have announced their partials; it covers the batch-1 latency setting of Appendix C.3 and the batched workloads alike) and
 * the two-launch pair (split-K kernel + combine pass) beyond that; the other two values force one of
 * them where the shape allows.  Both compute Eq. 1 / Eq. 2 over the same rows.  The single-launch
 * kernel is issued with programmatic stream serialisation: it starts with a grid-dependency wait (see
 * flux_plan_set_launch_overlap), so results never depend on it, and it lets the next such launch in
 * the stream be set up while it drains.  Its CTAs (one per SM) wait for one another when they merge
 * (bounded: about a second), so it expects to get the GPU's SMs while it runs; if other work -- another
 * stream's long kernel, a second launch of this kernel running at the same time -- keeps some of its
 * CTAs from starting for that long, the wait expires, FLUX_STATUS_WAIT_EXPIRED is raised and the
 * outputs of that launch are not valid.  Callers that run several decode streams on one GPU at once
 * select FLUX_DECODE_TWO_LAUNCH, whose kernels never wait for each other. */
#define FLUX_DECODE_AUTO          0
#define FLUX_DECODE_TWO_LAUNCH    1
#define FLUX_DECODE_SINGLE_LAUNCH 2
int flux_debug_decode_kernel(flux_plan *plan, int32_t which);

/* Exercises the give-up path of the kernels' bounded waits without any fault: launches one warp
 * that waits, with the same bounded wait the prefill kernel uses, on a barrier nothing arrives
 * at.  After limit_cycles SM clock cycles (1 .. 2e9) the wait runs out, the kernel sets
 * FLUX_STATUS_WAIT_EXPIRED and returns; flux_plan_status() then reports FLUX_E_DEVICE_TIMEOUT
 * and clears the word.  While the bit is set, prefill CTAs return at once without computing. */
int flux_debug_wait_probe(flux_plan *plan, int64_t limit_cycles, void *stream);

/* Number of kernels this plan has launched so far (host counter). */
int64_t flux_launch_count(const flux_plan *plan);

/* Message for the most recent failure on the calling thread ("" if none). */
const char *flux_last_error(void);

/* Library version, "major.minor". */
const char *flux_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FLUX_ATTN_H */
