// Entry points of libflux_attn.so: plan, workspace, hard routing, KV append and
// retention, status and dispatch records.  The attention kernels live in
// flux_decode.cu and flux_prefill*.cu.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "flux_internal.h"

namespace flux {

static thread_local char g_err[512] = "";

int fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return code;
}

int check_cuda(cudaError_t e, const char *what)
{
    if (e == cudaSuccess) return FLUX_OK;
    return fail(FLUX_E_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

int prof_begin(flux_plan *p, int kind, cudaStream_t st)
{
    if (!p->prof_ev || p->prof_n >= p->prof_cap) return -1;
    const int rec = p->prof_n++;
    p->prof_kind[rec] = (int8_t)kind;
    cudaEventRecord(p->prof_ev[2 * rec], st);
    return rec;
}

void prof_end(flux_plan *p, int rec, cudaStream_t st)
{
    if (rec >= 0) cudaEventRecord(p->prof_ev[2 * rec + 1], st);
}

static void prof_free(flux_plan *p)
{
    if (p->prof_ev) {
        for (int i = 0; i < 2 * p->prof_cap; ++i) cudaEventDestroy(p->prof_ev[i]);
        free(p->prof_ev);
        free(p->prof_kind);
    }
    p->prof_ev = nullptr;
    p->prof_kind = nullptr;
    p->prof_cap = p->prof_n = 0;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static int validate_config(const flux_config *c)
{
    if (!c) return fail(FLUX_E_INVALID_ARG, "config is NULL");
    if (c->head_dim != kHeadDim)
        return fail(FLUX_E_UNSUPPORTED_SHAPE, "head_dim %d unsupported (must be 128)", c->head_dim);
    if (c->n_layers < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1)
        return fail(FLUX_E_INVALID_ARG, "n_layers, n_q_heads, n_kv_heads must be >= 1");
    if (c->n_q_heads % c->n_kv_heads != 0)
        return fail(FLUX_E_UNSUPPORTED_SHAPE, "n_q_heads %d is not a multiple of n_kv_heads %d",
                    c->n_q_heads, c->n_kv_heads);
    if (c->n_q_heads / c->n_kv_heads > 16)
        return fail(FLUX_E_UNSUPPORTED_SHAPE, "more than 16 query heads per KV head");
    if (c->sink < 0 || c->window < 1)
        return fail(FLUX_E_INVALID_ARG, "need sink >= 0 and window >= 1");
    if (c->max_batch < 1 || c->max_batch > kMaxBatch)
        return fail(FLUX_E_CAPACITY, "max_batch must be in [1, %d]", kMaxBatch);
    if (c->max_context < 1 || (int64_t)c->max_context + 1 >= (1ll << 30))
        return fail(FLUX_E_CAPACITY, "max_context must be in [1, 2^30)");
    if ((int64_t)c->sink + c->window >= (1ll << 30))
        return fail(FLUX_E_CAPACITY, "sink + window too large");
    if (c->kv_layout != FLUX_KV_FULL && c->kv_layout != FLUX_KV_COMPACT_SA)
        return fail(FLUX_E_INVALID_ARG, "unknown kv_layout %d", c->kv_layout);
    if (!(c->softmax_scale >= 0.0f) || isinf(c->softmax_scale))
        return fail(FLUX_E_INVALID_ARG, "softmax_scale must be finite and >= 0");
    return FLUX_OK;
}

WorkspaceLayout workspace_layout(const flux_config &c)
{
    WorkspaceLayout w;
    const size_t A = 256;
    size_t off = 0;
    const int G = c.n_q_heads / c.n_kv_heads;
    const size_t B = (size_t)c.max_batch, L = (size_t)c.n_layers;
    w.status = off;       off = align_up(off + 64, A);
    w.debug = off;        off = align_up(off + B * 8 * sizeof(int32_t), A);
    w.sched = off;        off = align_up(off + (B + 4) * sizeof(int32_t), A);
    w.stage_mask = off;   off = align_up(off + B * L, A);
    w.stage_logits = off; off = align_up(off + B * L * 2 * sizeof(float), A);
    w.slots = ((int64_t)kDecMaxCtas + (int64_t)B * dec_head_groups(c.n_kv_heads)) * kDecWarps;
    w.part_o = off;       off = align_up(off + (size_t)w.slots * G * kHeadDim * sizeof(float), A);
    w.part_ml = off;      off = align_up(off + (size_t)w.slots * G * 2 * sizeof(float), A);
    w.host_q = off;       off = align_up(off + B * c.n_q_heads * kRowBytes, A);
    w.host_k = off;       off = align_up(off + B * c.n_kv_heads * kRowBytes, A);
    w.host_v = off;       off = align_up(off + B * c.n_kv_heads * kRowBytes, A);
    w.host_o = off;       off = align_up(off + B * c.n_q_heads * kRowBytes, A);
    w.router = off;       off = align_up(off + ((size_t)2 * c.n_q_heads * kHeadDim + 6 * kRouterMaxWidth) * sizeof(float), A);
    w.router_sync = off;  off = align_up(off + 8 * sizeof(uint32_t), A);
    w.tickets = off;      off = align_up(off + 2 * (size_t)kDecFusedMaxBatch * c.n_kv_heads * sizeof(uint32_t), A);
    w.push_ticket = off;  off = align_up(off + 8 * sizeof(uint32_t), A);
    w.total = off;
    return w;
}

static bool aligned16(const void *p) { return (((uintptr_t)p) & 15u) == 0; }

// true if p is device-accessible global memory (device or managed allocation)
static bool is_device_ptr(const void *p)
{
    cudaPointerAttributes a;
    cudaError_t e = cudaPointerGetAttributes(&a, p);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return a.type == cudaMemoryTypeDevice || a.type == cudaMemoryTypeManaged;
}

// device-side address of a pinned (page-locked, mapped) host buffer, or NULL for any other memory
static const void *mapped_host_ptr(const void *p)
{
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
}

static int need_plan(flux_plan *p, bool need_ws)
{
    if (!p) return fail(FLUX_E_INVALID_ARG, "plan is NULL");
    if (need_ws && !p->ws) return fail(FLUX_E_WORKSPACE, "no workspace set on the plan");
    return FLUX_OK;
}

static int need_mask(flux_plan *p, int layer)
{
    if (layer < 0 || layer >= p->cfg.n_layers)
        return fail(FLUX_E_INVALID_ARG, "layer %d outside [0, %d)", layer, p->cfg.n_layers);
    if (!p->d_mask)
        return fail(FLUX_E_INVALID_ARG, "flux_router_apply has not been called on this plan");
    return FLUX_OK;
}

// ---------------------------------------------------------------------------------------------
// small kernels
// ---------------------------------------------------------------------------------------------

// Hard routing (Sec. 3.1): mask = (pi_FA >= pi_SA), or a validated copy of a given mask.
__global__ void router_kernel(const float *__restrict__ logits, const uint8_t *__restrict__ mask_in,
                              uint8_t *__restrict__ mask_out, int n, uint32_t *status)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    if (mask_in) {
        uint8_t m = mask_in[i];
        if (m > 1) {
            atomicOr(status, FLUX_STATUS_BAD_MASK);
            m = 1;  // an unreadable decision falls back to the dense mode
        }
        mask_out[i] = m;
    } else {
        float fa = logits[2 * i], sa = logits[2 * i + 1];
        if (isnan(fa) || isnan(sa)) {
            atomicOr(status, FLUX_STATUS_NAN_LOGIT);
            mask_out[i] = 1;
        } else {
            mask_out[i] = (fa >= sa) ? 1 : 0;
        }
    }
}

// Row of the cache that holds position `pos`.
__device__ __forceinline__ int64_t cache_row(int pos, bool compact_sa, int S, int W)
{
    if (!compact_sa || pos < S) return pos;
    return (int64_t)S + (pos - S) % W;
}

// One token per request: 16 bytes per thread, K row then V row.
__global__ void kv_append_kernel(const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new,
                                 void *const *__restrict__ k_caches, void *const *__restrict__ v_caches,
                                 const int32_t *__restrict__ pos, const uint8_t *__restrict__ mask,
                                 int L, int layer, int row_u4, int S, int W, int layout,
                                 int max_context, uint32_t *status)
{
    const int b = blockIdx.x;
    const int p = pos[b];
    if (p < 0) return;
    if (p >= max_context) {
        if (threadIdx.x == 0) atomicOr(status, FLUX_STATUS_BAD_LENGTH);
        return;
    }
    const bool compact = (layout == FLUX_KV_COMPACT_SA) && (mask[b * L + layer] == 0);
    const int64_t row = cache_row(p, compact, S, W);
    uint4 *kd = (uint4 *)k_caches[b] + row * row_u4;
    uint4 *vd = (uint4 *)v_caches[b] + row * row_u4;
    for (int i = threadIdx.x; i < row_u4; i += blockDim.x) {
        kd[i] = k_new[(int64_t)b * row_u4 + i];
        vd[i] = v_new[(int64_t)b * row_u4 + i];
    }
}

// Prefill -> cache hand-off: copy the rows decode will need (see flux_kv_retain).
__global__ void kv_retain_kernel(const uint4 *__restrict__ k_src, const uint4 *__restrict__ v_src,
                                 uint4 *__restrict__ k_dst, uint4 *__restrict__ v_dst, int n,
                                 const uint8_t *__restrict__ mask, int L, int layer, int req,
                                 int row_u4, int S, int W, int layout, int copy_identity)
{
    const bool compact = (layout == FLUX_KV_COMPACT_SA) && (mask[req * L + layer] == 0);
    if (!compact && !copy_identity) return;  // source already is the cache
    // kept rows: [0, a1) and [b0, n); for a full copy a1 = n and the second range is empty
    const int a1 = compact ? min(S, n) : n;
    const int b0 = compact ? min(n, max(S, n - W)) : n;
    const int n_rows = a1 + (n - b0);
    for (int r = blockIdx.x; r < n_rows; r += gridDim.x) {
        const int p = r < a1 ? r : b0 + (r - a1);
        const int64_t row = cache_row(p, compact, S, W);
        for (int i = threadIdx.x; i < row_u4; i += blockDim.x) {
            k_dst[row * row_u4 + i] = k_src[(int64_t)p * row_u4 + i];
            v_dst[row * row_u4 + i] = v_src[(int64_t)p * row_u4 + i];
        }
    }
}

// flux_attn_decode_host with pinned (device-mapped) activations: one launch reads the request's new
// K, V rows and its query rows straight from host memory, each byte once -- the K, V rows go into
// the caches like kv_append_kernel does, the query rows into device staging (the decode kernel
// re-reads them from every CTA, which must not cross the bus).
// Issued with programmatic stream serialisation when launch overlap is on: the reads from host memory (the slow part:
// they cross the bus) are done before the grid-dependency wait, into registers, while the previous decode launch is
// still running; everything the kernel writes -- the query staging that launch reads, the cache rows -- comes after it.
constexpr int kIngestQ = 8, kIngestKV = 2;   // 16-byte pieces per thread held in registers across the wait
__global__ void __launch_bounds__(256)
host_ingest_kernel(const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new,
                   const uint4 *__restrict__ q_host, uint4 *__restrict__ q_stage, int q_u4,
                   void *const *__restrict__ k_caches, void *const *__restrict__ v_caches,
                   const int32_t *__restrict__ pos, const uint8_t *__restrict__ mask,
                   int L, int layer, int row_u4, int S, int W, int layout,
                   int max_context, uint32_t *status)
{
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    uint4 qr[kIngestQ], kr[kIngestKV], vr[kIngestKV];
#pragma unroll
    for (int j = 0; j < kIngestQ; ++j)
        if (tid + j * nt < q_u4) qr[j] = q_host[(int64_t)b * q_u4 + tid + j * nt];
#pragma unroll
    for (int j = 0; j < kIngestKV; ++j)
        if (tid + j * nt < row_u4) {
            kr[j] = k_new[(int64_t)b * row_u4 + tid + j * nt];
            vr[j] = v_new[(int64_t)b * row_u4 + tid + j * nt];
        }
    const int p = pos[b];
    const bool compact = (layout == FLUX_KV_COMPACT_SA) && (mask[b * L + layer] == 0);
    uint4 *kc = (uint4 *)k_caches[b], *vc = (uint4 *)v_caches[b];
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
#pragma unroll
    for (int j = 0; j < kIngestQ; ++j)
        if (tid + j * nt < q_u4) q_stage[(int64_t)b * q_u4 + tid + j * nt] = qr[j];
    for (int i = tid + kIngestQ * nt; i < q_u4; i += nt) q_stage[(int64_t)b * q_u4 + i] = q_host[(int64_t)b * q_u4 + i];
    if (p < 0) return;
    if (p >= max_context) {
        if (tid == 0) atomicOr(status, FLUX_STATUS_BAD_LENGTH);
        return;
    }
    const int64_t row = cache_row(p, compact, S, W);
    uint4 *kd = kc + row * row_u4, *vd = vc + row * row_u4;
#pragma unroll
    for (int j = 0; j < kIngestKV; ++j)
        if (tid + j * nt < row_u4) {
            kd[tid + j * nt] = kr[j];
            vd[tid + j * nt] = vr[j];
        }
    for (int i = tid + kIngestKV * nt; i < row_u4; i += nt) {
        kd[i] = k_new[(int64_t)b * row_u4 + i];
        vd[i] = v_new[(int64_t)b * row_u4 + i];
    }
}

int launch_router(flux_plan *p, const float *d_logits, const uint8_t *d_mask_in, int B,
                  uint8_t *d_mask_out, cudaStream_t st)
{
    const int n = B * p->cfg.n_layers;
    uint32_t *status = (uint32_t *)((char *)p->ws + p->lay.status);
    router_kernel<<<(n + 127) / 128, 128, 0, st>>>(d_logits, d_mask_in, d_mask_out, n, status);
    p->launches++;
    return check_cuda(cudaGetLastError(), "router kernel launch");
}

int launch_kv_append(flux_plan *p, int layer, int B, const void *k_new, const void *v_new,
                     void *const *k_caches, void *const *v_caches, const int32_t *pos,
                     cudaStream_t st)
{
    const flux_config &c = p->cfg;
    const int row_u4 = c.n_kv_heads * kRowBytes / 16;
    uint32_t *status = (uint32_t *)((char *)p->ws + p->lay.status);
    kv_append_kernel<<<B, 128, 0, st>>>((const uint4 *)k_new, (const uint4 *)v_new, k_caches,
                                        v_caches, pos, p->d_mask, c.n_layers, layer, row_u4,
                                        c.sink, c.window, c.kv_layout, c.max_context, status);
    p->launches++;
    return check_cuda(cudaGetLastError(), "kv_append kernel launch");
}

int launch_kv_retain(flux_plan *p, int layer, int req, const void *k_src, const void *v_src,
                     int n, void *k_cache, void *v_cache, cudaStream_t st)
{
    const flux_config &c = p->cfg;
    const int row_u4 = c.n_kv_heads * kRowBytes / 16;
    const int copy_identity = (k_src != k_cache || v_src != v_cache) ? 1 : 0;
    int grid = n < 1 ? 1 : (n > p->dev.n_sms * 8 ? p->dev.n_sms * 8 : n);
    kv_retain_kernel<<<grid, 128, 0, st>>>((const uint4 *)k_src, (const uint4 *)v_src,
                                           (uint4 *)k_cache, (uint4 *)v_cache, n, p->d_mask,
                                           c.n_layers, layer, req, row_u4, c.sink, c.window,
                                           c.kv_layout, copy_identity);
    p->launches++;
    return check_cuda(cudaGetLastError(), "kv_retain kernel launch");
}

}  // namespace flux

using namespace flux;

// ---------------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------------

extern "C" {

const char *flux_last_error(void) { return g_err; }
const char *flux_version(void) { return "0.1"; }

int flux_workspace_size(const flux_config *cfg, size_t *bytes_out)
{
    int rc = validate_config(cfg);
    if (rc) return rc;
    if (!bytes_out) return fail(FLUX_E_INVALID_ARG, "bytes_out is NULL");
    *bytes_out = workspace_layout(*cfg).total;
    return FLUX_OK;
}

int flux_plan_create(const flux_config *cfg, flux_plan **plan)
{
    if (plan) *plan = nullptr;
    int rc = validate_config(cfg);
    if (rc) return rc;
    if (!plan) return fail(FLUX_E_INVALID_ARG, "plan out-pointer is NULL");
    int dev = 0;
    rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
    if (rc) return rc;
    flux_plan *p = new (std::nothrow) flux_plan();
    if (!p) return fail(FLUX_E_INVALID_ARG, "out of host memory");
    p->cfg = *cfg;
    p->G = cfg->n_q_heads / cfg->n_kv_heads;
    p->scale = cfg->softmax_scale > 0.0f ? cfg->softmax_scale : 1.0f / sqrtf((float)cfg->head_dim);
    p->scale_log2 = p->scale * 1.4426950408889634f;
    p->ws = nullptr;
    p->ws_bytes = 0;
    p->lay = workspace_layout(*cfg);
    p->d_mask = nullptr;
    p->mask_B = 0;
    p->launches = 0;
    p->debug_records = 0;
    p->touch = nullptr;
    p->touch_words = 0;
    p->prof_ev = nullptr;
    p->prof_kind = nullptr;
    p->prof_cap = p->prof_n = 0;
    cudaError_t e = cudaDeviceGetAttribute(&p->dev.n_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess)
        e = cudaDeviceGetAttribute(&p->dev.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e == cudaSuccess)
        e = cudaDeviceGetAttribute(&p->dev.cc_major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) {
        delete p;
        return check_cuda(e, "cudaDeviceGetAttribute");
    }
    if (p->dev.cc_major != 10) {
        int cc = p->dev.cc_major;
        delete p;
        return fail(FLUX_E_CUDA, "this library is built for sm_100a only (device is sm_%d0)", cc);
    }
    p->dec_ctas = p->dev.n_sms < kDecMaxCtas ? p->dev.n_sms : kDecMaxCtas;
    p->decode_kernel = FLUX_DECODE_AUTO;
    p->launch_overlap = 0;
    rc = decode_setup(p);
    if (!rc) rc = decode_fused_setup(p);
    if (!rc) rc = prefill_setup(p);
    if (!rc) rc = router_setup(p);
    if (rc) {
        delete p;
        return rc;
    }
    *plan = p;
    return FLUX_OK;
}

int flux_plan_destroy(flux_plan *plan)
{
    if (plan) prof_free(plan);
    delete plan;
    return FLUX_OK;
}

int flux_plan_set_workspace(flux_plan *plan, void *workspace, size_t bytes)
{
    int rc = need_plan(plan, false);
    if (rc) return rc;
    if (!workspace || (((uintptr_t)workspace) & 255u))
        return fail(FLUX_E_INVALID_ARG, "workspace must be a 256-byte aligned device pointer");
    if (bytes < plan->lay.total)
        return fail(FLUX_E_WORKSPACE, "workspace of %zu bytes is smaller than the %zu needed", bytes,
                    plan->lay.total);
    plan->ws = workspace;
    plan->ws_bytes = bytes;
    return FLUX_OK;
}

int flux_router_apply(flux_plan *plan, const float *logits, const uint8_t *mask_or_null, int32_t B,
                      uint8_t *mask_out, void *stream)
{
    int rc = need_plan(plan, true);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const flux_config &c = plan->cfg;
    if (B < 1 || B > c.max_batch) return fail(FLUX_E_CAPACITY, "B=%d outside [1, %d]", B, c.max_batch);
    if (!mask_out) return fail(FLUX_E_INVALID_ARG, "mask_out is NULL");
    if (!logits && !mask_or_null) return fail(FLUX_E_INVALID_ARG, "neither logits nor a mask given");
    const size_t n = (size_t)B * c.n_layers;
    const float *d_logits = nullptr;
    const uint8_t *d_mask_in = nullptr;
    if (mask_or_null) {
        if (is_device_ptr(mask_or_null)) {
            d_mask_in = mask_or_null;
        } else {
            for (size_t i = 0; i < n; ++i)
                if (mask_or_null[i] > 1)
                    return fail(FLUX_E_INVALID_ARG, "mask byte %zu is %d, not 0 or 1", i,
                                (int)mask_or_null[i]);
            uint8_t *stg = (uint8_t *)plan->ws + plan->lay.stage_mask;
            rc = check_cuda(cudaMemcpyAsync(stg, mask_or_null, n, cudaMemcpyHostToDevice, st),
                            "mask upload");
            if (rc) return rc;
            d_mask_in = stg;
        }
    } else {
        if (is_device_ptr(logits)) {
            if (!aligned16(logits)) return fail(FLUX_E_INVALID_ARG, "logits not 16-byte aligned");
            d_logits = logits;
        } else {
            for (size_t i = 0; i < 2 * n; ++i)
                if (isnan(logits[i])) return fail(FLUX_E_INVALID_ARG, "routing logit %zu is NaN", i);
            float *stg = (float *)((char *)plan->ws + plan->lay.stage_logits);
            rc = check_cuda(cudaMemcpyAsync(stg, logits, 2 * n * sizeof(float),
                                            cudaMemcpyHostToDevice, st), "logits upload");
            if (rc) return rc;
            d_logits = stg;
        }
    }
    rc = launch_router(plan, d_logits, d_mask_in, B, mask_out, st);
    if (rc) return rc;
    plan->d_mask = mask_out;
    plan->mask_B = B;
    return FLUX_OK;
}

int flux_router_forward(flux_plan *plan, const flux_router_weights *w, const void *q_first, int32_t n_first,
                        const void *q_last, int32_t n_last, float *logits_out, void *stream)
{
    int rc = need_plan(plan, true);
    if (rc) return rc;
    if (!w) return fail(FLUX_E_INVALID_ARG, "router weights are NULL");
    if (!q_first || !q_last || !logits_out) return fail(FLUX_E_INVALID_ARG, "NULL tensor pointer");
    if (n_first < 1 || n_last < 1) return fail(FLUX_E_INVALID_ARG, "a pooled segment needs at least one token");
    if (w->enc_dim < 8 || w->head_hidden < 8 || (w->enc_dim & 7) || (w->head_hidden & 7))
        return fail(FLUX_E_UNSUPPORTED_SHAPE, "router widths %d / %d must be multiples of 8", w->enc_dim, w->head_hidden);
    if (w->enc_dim > kRouterMaxWidth || w->head_hidden > kRouterMaxWidth)
        return fail(FLUX_E_CAPACITY, "router widths %d / %d exceed %d", w->enc_dim, w->head_hidden, kRouterMaxWidth);
    const void *ptrs[] = {w->w_enc1, w->b_enc1, w->w_enc2, w->b_enc2, w->w_head1, w->b_head1, w->w_head2, w->b_head2};
    for (const void *ptr : ptrs)
        if (!ptr || !aligned16(ptr)) return fail(FLUX_E_INVALID_ARG, "router weight pointer NULL or not 16-byte aligned");
    if (!aligned16(q_first) || !aligned16(q_last)) return fail(FLUX_E_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    if (((uintptr_t)logits_out & 7u) != 0) return fail(FLUX_E_INVALID_ARG, "logits_out must be 8-byte aligned");
    if (!is_device_ptr(logits_out)) return fail(FLUX_E_INVALID_ARG, "logits_out must be device memory");
    return launch_router_frontend(plan, w, q_first, n_first, q_last, n_last, logits_out, (cudaStream_t)stream);
}

int flux_attn_prefill(flux_plan *plan, int32_t layer, int32_t req, const void *q, const void *k,
                      const void *v, int32_t q_start, int32_t Nq, void *out, void *stream)
{
    int rc = need_plan(plan, true);
    if (rc) return rc;
    rc = need_mask(plan, layer);
    if (rc) return rc;
    if (req < 0 || req >= plan->mask_B)
        return fail(FLUX_E_INVALID_ARG, "request %d outside the routed batch of %d", req, plan->mask_B);
    if (Nq < 0 || q_start < 0) return fail(FLUX_E_INVALID_ARG, "negative q_start or Nq");
    if ((int64_t)q_start + Nq > plan->cfg.max_context)
        return fail(FLUX_E_CAPACITY, "q_start + Nq = %lld exceeds max_context %d",
                    (long long)q_start + Nq, plan->cfg.max_context);
    if (Nq == 0) return FLUX_OK;
    if (!q || !k || !v || !out) return fail(FLUX_E_INVALID_ARG, "NULL tensor pointer");
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
        return fail(FLUX_E_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    return launch_prefill(plan, layer, req, q, k, v, q_start, Nq, out, (cudaStream_t)stream);
}

int flux_attn_prefill_blocks(flux_plan *plan, const void *q, const void *k, const void *v, int32_t q_start,
                             int32_t Nq, const uint8_t *block_mask, int32_t n_kv_blocks, void *out, void *stream)
{
    int rc = need_plan(plan, true);
    if (rc) return rc;
    if (Nq < 0 || q_start < 0) return fail(FLUX_E_INVALID_ARG, "negative q_start or Nq");
    if (q_start % 64) return fail(FLUX_E_INVALID_ARG, "q_start must be a multiple of the block size (64)");
    if ((int64_t)q_start + Nq > plan->cfg.max_context)
        return fail(FLUX_E_CAPACITY, "q_start + Nq = %lld exceeds max_context %d",
                    (long long)q_start + Nq, plan->cfg.max_context);
    if (Nq == 0) return FLUX_OK;
    if ((int64_t)n_kv_blocks * 64 < (int64_t)q_start + Nq)
        return fail(FLUX_E_INVALID_ARG, "block mask rows of %d blocks do not cover %lld positions", n_kv_blocks,
                    (long long)q_start + Nq);
    if (!q || !k || !v || !out || !block_mask) return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
        return fail(FLUX_E_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    return launch_prefill_blocks(plan, q, k, v, q_start, Nq, block_mask, n_kv_blocks, out, (cudaStream_t)stream);
}

int flux_debug_touched(flux_plan *plan, uint32_t *bitmap, int32_t words_per_request)
{
    int rc = need_plan(plan, false);
    if (rc) return rc;
    if (bitmap && (words_per_request < 1 || (int64_t)words_per_request * 32 < plan->cfg.max_context))
        return fail(FLUX_E_INVALID_ARG, "the bitmap needs one bit per position up to max_context");
    plan->touch = bitmap;
    plan->touch_words = bitmap ? words_per_request : 0;
    return FLUX_OK;
}

int flux_debug_wait_probe(flux_plan *plan, int64_t limit_cycles, void *stream)
{
    int rc = need_plan(plan, true);
    if (rc) return rc;
    if (limit_cycles < 1 || limit_cycles > 2000000000ll)
        return fail(FLUX_E_INVALID_ARG, "limit_cycles must be in [1, 2e9]");
    return launch_wait_probe(plan, limit_cycles, (cudaStream_t)stream);
}

int flux_plan_set_launch_overlap(flux_plan *plan, int32_t on)
{
    int rc = need_plan(plan, false);
    if (rc) return rc;
    plan->launch_overlap = on ? 1 : 0;
    return FLUX_OK;
}

int flux_debug_decode_kernel(flux_plan *plan, int32_t which)
{
    int rc = need_plan(plan, false);
    if (rc) return rc;
    if (which < FLUX_DECODE_AUTO || which > FLUX_DECODE_SINGLE_LAUNCH)
        return fail(FLUX_E_INVALID_ARG, "unknown decode kernel selector %d", which);
    plan->decode_kernel = which;
    return FLUX_OK;
}

int flux_kv_retain(flux_plan *plan, int32_t layer, int32_t req, const void *k_src, const void *v_src,
                   int32_t n, void *k_cache, void *v_cache, void *stream)
{
    int rc = need_plan(plan, true);
    if (rc) return rc;
    rc = need_mask(plan, layer);
    if (rc) return rc;
    if (req < 0 || req >= plan->mask_B)
        return fail(FLUX_E_INVALID_ARG, "request %d outside the routed batch of %d", req, plan->mask_B);
    if (n < 0 || n > plan->cfg.max_context)
        return fail(FLUX_E_CAPACITY, "n=%d outside [0, max_context=%d]", n, plan->cfg.max_context);
    if (n == 0) return FLUX_OK;
    if (!k_src || !v_src || !k_cache || !v_cache) return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    if (!aligned16(k_src) || !aligned16(v_src) || !aligned16(k_cache) || !aligned16(v_cache))
        return fail(FLUX_E_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    return launch_kv_retain(plan, layer, req, k_src, v_src, n, k_cache, v_cache,
                            (cudaStream_t)stream);
}

static int check_batch_call(flux_plan *plan, int layer, int B)
{
    int rc = need_plan(plan, true);
    if (rc) return rc;
    rc = need_mask(plan, layer);
    if (rc) return rc;
    if (B < 1 || B > plan->mask_B)
        return fail(FLUX_E_CAPACITY, "B=%d outside [1, routed batch %d]", B, plan->mask_B);
    return FLUX_OK;
}

int flux_kv_append(flux_plan *plan, int32_t layer, int32_t B, const void *k_new, const void *v_new,
                   void *const *k_caches, void *const *v_caches, const int32_t *pos, void *stream)
{
    int rc = check_batch_call(plan, layer, B);
    if (rc) return rc;
    if (!k_new || !v_new || !k_caches || !v_caches || !pos)
        return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    if (!aligned16(k_new) || !aligned16(v_new))
        return fail(FLUX_E_INVALID_ARG, "k_new / v_new must be 16-byte aligned");
    return launch_kv_append(plan, layer, B, k_new, v_new, k_caches, v_caches, pos,
                            (cudaStream_t)stream);
}

int flux_attn_decode(flux_plan *plan, int32_t layer, int32_t B, const void *q,
                     const void *const *k_caches, const void *const *v_caches,
                     const int32_t *ctx_len, void *out, void *stream)
{
    int rc = check_batch_call(plan, layer, B);
    if (rc) return rc;
    if (!q || !k_caches || !v_caches || !ctx_len || !out)
        return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    if (!aligned16(q) || !aligned16(out))
        return fail(FLUX_E_INVALID_ARG, "q / out must be 16-byte aligned");
    return launch_decode(plan, layer, B, q, k_caches, v_caches, ctx_len, out, (cudaStream_t)stream);
}

int flux_attn_decode_partial(flux_plan *plan, int32_t layer, int32_t B, const void *q, const void *const *k_caches,
                             const void *const *v_caches, const int32_t *ctx_len, const int32_t *key_begin,
                             const int32_t *key_end, float *part_o, float *part_ml, void *stream)
{
    int rc = check_batch_call(plan, layer, B);
    if (rc) return rc;
    if (!q || !k_caches || !v_caches || !ctx_len || !key_begin || !key_end || !part_o || !part_ml)
        return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    if (!aligned16(q) || !aligned16(part_o) || (((uintptr_t)part_ml) & 7u))
        return fail(FLUX_E_INVALID_ARG, "q / part_o must be 16-byte aligned, part_ml 8-byte aligned");
    if (!is_device_ptr(key_begin) || !is_device_ptr(key_end) || !is_device_ptr(part_o) || !is_device_ptr(part_ml))
        return fail(FLUX_E_INVALID_ARG, "key ranges and partial outputs must be device memory");
    DecPartial part = {key_begin, key_end, part_o, part_ml, {}};
    part.push.world = 0;
    return launch_decode(plan, layer, B, q, k_caches, v_caches, ctx_len, nullptr, (cudaStream_t)stream, nullptr, nullptr,
                         nullptr, &part);
}

int flux_attn_decode_partial_push(flux_plan *plan, int32_t layer, int32_t B, const void *q, const void *const *k_caches,
                                  const void *const *v_caches, const int32_t *ctx_len, const int32_t *key_begin,
                                  const int32_t *key_end, const flux_peer_set *peers, uint32_t seq, void *stream)
{
    int rc = check_batch_call(plan, layer, B);
    if (rc) return rc;
    if (!q || !k_caches || !v_caches || !ctx_len || !key_begin || !key_end || !peers)
        return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    if (!aligned16(q)) return fail(FLUX_E_INVALID_ARG, "q must be 16-byte aligned");
    if (!is_device_ptr(key_begin) || !is_device_ptr(key_end))
        return fail(FLUX_E_INVALID_ARG, "key ranges must be device memory");
    if (peers->world < 1 || peers->world > kMaxPeers || peers->rank < 0 || peers->rank >= peers->world)
        return fail(FLUX_E_INVALID_ARG, "world=%d (1..%d) / rank=%d", peers->world, kMaxPeers, peers->rank);
    if (seq == 0) return fail(FLUX_E_INVALID_ARG, "seq must not be 0 (the value of a cleared flag array)");
    DecPartial part = {key_begin, key_end, nullptr, nullptr, {}};
    part.push.world = peers->world;
    part.push.rank = peers->rank;
    part.push.seq = seq;
    for (int p = 0; p < peers->world; ++p) {
        if (!peers->gather_o[p] || !peers->gather_ml[p] || !peers->flags[p])
            return fail(FLUX_E_INVALID_ARG, "peer %d: NULL pointer", p);
        if (!aligned16(peers->gather_o[p]) || (((uintptr_t)peers->gather_ml[p]) & 7u) || (((uintptr_t)peers->flags[p]) & 3u))
            return fail(FLUX_E_INVALID_ARG, "peer %d: gather_o must be 16-byte, gather_ml 8-byte, flags 4-byte aligned", p);
        part.push.o[p] = peers->gather_o[p];
        part.push.ml[p] = peers->gather_ml[p];
        part.push.flags[p] = peers->flags[p];
    }
    return launch_decode(plan, layer, B, q, k_caches, v_caches, ctx_len, nullptr, (cudaStream_t)stream, nullptr, nullptr,
                         nullptr, &part);
}

int flux_attn_combine_wait(flux_plan *plan, int32_t B, int32_t world, const float *gather_o, const float *gather_ml,
                           const uint32_t *flags, uint32_t seq, int64_t wait_cycles, void *out, void *stream)
{
    int rc = need_plan(plan, true);
    if (rc) return rc;
    if (B < 1 || B > plan->cfg.max_batch) return fail(FLUX_E_CAPACITY, "B=%d outside [1, %d]", B, plan->cfg.max_batch);
    if (world < 1 || world > kMaxPeers) return fail(FLUX_E_INVALID_ARG, "world=%d outside [1, %d]", world, kMaxPeers);
    if (!gather_o || !gather_ml || !flags || !out) return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    if (!aligned16(gather_o) || !aligned16(out) || (((uintptr_t)gather_ml) & 7u) || (((uintptr_t)flags) & 3u))
        return fail(FLUX_E_INVALID_ARG, "gather_o / out must be 16-byte, gather_ml 8-byte, flags 4-byte aligned");
    if (seq == 0) return fail(FLUX_E_INVALID_ARG, "seq must not be 0");
    if (wait_cycles < 0 || wait_cycles > 4000000000ll) return fail(FLUX_E_INVALID_ARG, "wait_cycles outside [0, 4e9]");
    return launch_combine_sets(plan, gather_o, gather_ml, world, B * plan->cfg.n_q_heads, out, (cudaStream_t)stream, flags, seq,
                               wait_cycles ? wait_cycles : 2000000000ll);
}

int flux_attn_combine(flux_plan *plan, int32_t B, int32_t n_sets, const float *part_o, const float *part_ml, void *out,
                      void *stream)
{
    int rc = need_plan(plan, false);
    if (rc) return rc;
    if (B < 1 || B > plan->cfg.max_batch) return fail(FLUX_E_CAPACITY, "B=%d outside [1, %d]", B, plan->cfg.max_batch);
    if (n_sets < 1 || n_sets > 1024) return fail(FLUX_E_INVALID_ARG, "n_sets=%d outside [1, 1024]", n_sets);
    if (!part_o || !part_ml || !out) return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    if (!aligned16(part_o) || !aligned16(out) || (((uintptr_t)part_ml) & 7u))
        return fail(FLUX_E_INVALID_ARG, "part_o / out must be 16-byte aligned, part_ml 8-byte aligned");
    return launch_combine_sets(plan, part_o, part_ml, n_sets, B * plan->cfg.n_q_heads, out, (cudaStream_t)stream);
}

int flux_attn_decode_heads(flux_plan *plan, int32_t B, const void *q, const void *const *k_caches,
                           const void *const *v_caches, const int32_t *ctx_len, const uint8_t *head_mask,
                           void *out, void *stream)
{
    int rc = need_plan(plan, true);
    if (rc) return rc;
    if (B < 1 || B > plan->cfg.max_batch) return fail(FLUX_E_CAPACITY, "B=%d outside [1, %d]", B, plan->cfg.max_batch);
    if (plan->cfg.kv_layout != FLUX_KV_FULL)
        return fail(FLUX_E_UNSUPPORTED_SHAPE, "head-level modes need the full cache layout (heads of a layer share its rows)");
    if (!q || !k_caches || !v_caches || !ctx_len || !head_mask || !out)
        return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    if (!is_device_ptr(head_mask)) return fail(FLUX_E_INVALID_ARG, "head_mask must be device memory");
    if (!aligned16(q) || !aligned16(out)) return fail(FLUX_E_INVALID_ARG, "q / out must be 16-byte aligned");
    return launch_decode(plan, 0, B, q, k_caches, v_caches, ctx_len, out, (cudaStream_t)stream, nullptr, nullptr,
                         head_mask);
}

int flux_attn_decode_step(flux_plan *plan, int32_t layer, int32_t B, const void *q, const void *k_new,
                          const void *v_new, void *const *k_caches, void *const *v_caches,
                          const int32_t *ctx_len, void *out, void *stream)
{
    int rc = check_batch_call(plan, layer, B);
    if (rc) return rc;
    if (!q || !k_new || !v_new || !k_caches || !v_caches || !ctx_len || !out)
        return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    if (!aligned16(q) || !aligned16(out) || !aligned16(k_new) || !aligned16(v_new))
        return fail(FLUX_E_INVALID_ARG, "q / k_new / v_new / out must be 16-byte aligned");
    return launch_decode(plan, layer, B, q, (const void *const *)k_caches, (const void *const *)v_caches, ctx_len,
                         out, (cudaStream_t)stream, k_new, v_new);
}

int flux_attn_decode_host(flux_plan *plan, int32_t layer, int32_t B, const void *q_host,
                          const void *k_new_host, const void *v_new_host, void *const *k_caches,
                          void *const *v_caches, const int32_t *pos, const int32_t *ctx_len,
                          void *out_host, void *stream)
{
    int rc = check_batch_call(plan, layer, B);
    if (rc) return rc;
    if (!q_host || !k_new_host || !v_new_host || !k_caches || !v_caches || !pos || !ctx_len ||
        !out_host)
        return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    cudaStream_t st = (cudaStream_t)stream;
    const flux_config &c = plan->cfg;
    char *ws = (char *)plan->ws;
    void *dq = ws + plan->lay.host_q, *dk = ws + plan->lay.host_k, *dv = ws + plan->lay.host_v,
         *dout = ws + plan->lay.host_o;
    const size_t qb = (size_t)B * c.n_q_heads * kRowBytes, kb = (size_t)B * c.n_kv_heads * kRowBytes;
    // Pinned host buffers are mapped into the device's address space: the kernels then read the
    // inputs and write the result in place (three launches, no copy operations in between).
    const void *mq = mapped_host_ptr(q_host), *mk = mapped_host_ptr(k_new_host), *mv = mapped_host_ptr(v_new_host);
    void *mo = const_cast<void *>(mapped_host_ptr(out_host));
    if (mq && mk && mv && mo && aligned16(mq) && aligned16(mk) && aligned16(mv) && aligned16(mo)) {
        const int row_u4 = c.n_kv_heads * kRowBytes / 16;
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3((unsigned)B);
        lc.blockDim = dim3(256);
        lc.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = attr;
        lc.numAttrs = plan->launch_overlap ? 1 : 0;   // same promise as for the decode launch (flux_plan_set_launch_overlap)
        rc = check_cuda(cudaLaunchKernelEx(&lc, host_ingest_kernel, (const uint4 *)mk, (const uint4 *)mv, (const uint4 *)mq,
                                           (uint4 *)dq, c.n_q_heads * kRowBytes / 16, (void *const *)k_caches,
                                           (void *const *)v_caches, pos, plan->d_mask, c.n_layers, layer, row_u4, c.sink,
                                           c.window, c.kv_layout, c.max_context, (uint32_t *)(ws + plan->lay.status)),
                        "host ingest kernel launch");
        plan->launches++;
        if (!rc)
            rc = launch_decode(plan, layer, B, dq, (const void *const *)k_caches, (const void *const *)v_caches,
                               ctx_len, mo, st);
        return rc;
    }
    rc = check_cuda(cudaMemcpyAsync(dq, q_host, qb, cudaMemcpyHostToDevice, st), "q upload");
    if (!rc) rc = check_cuda(cudaMemcpyAsync(dk, k_new_host, kb, cudaMemcpyHostToDevice, st), "k upload");
    if (!rc) rc = check_cuda(cudaMemcpyAsync(dv, v_new_host, kb, cudaMemcpyHostToDevice, st), "v upload");
    if (!rc) rc = launch_kv_append(plan, layer, B, dk, dv, k_caches, v_caches, pos, st);
    if (!rc)
        rc = launch_decode(plan, layer, B, dq, (const void *const *)k_caches,
                           (const void *const *)v_caches, ctx_len, dout, st);
    if (!rc) rc = check_cuda(cudaMemcpyAsync(out_host, dout, qb, cudaMemcpyDeviceToHost, st), "out download");
    return rc;
}

int flux_attn_prefill_host(flux_plan *plan, int32_t layer, int32_t req, const void *q_host,
                           void *q_dev, const void *k, const void *v, int32_t q_start, int32_t Nq,
                           void *out_dev, void *out_host, void *stream)
{
    int rc = need_plan(plan, true);
    if (rc) return rc;
    if (Nq < 0) return fail(FLUX_E_INVALID_ARG, "negative Nq");
    if (Nq == 0) return FLUX_OK;
    if (!q_host || !q_dev || !out_dev || !out_host) return fail(FLUX_E_INVALID_ARG, "NULL pointer");
    cudaStream_t st = (cudaStream_t)stream;
    const size_t qb = (size_t)Nq * plan->cfg.n_q_heads * kRowBytes;
    rc = check_cuda(cudaMemcpyAsync(q_dev, q_host, qb, cudaMemcpyHostToDevice, st), "q upload");
    if (!rc) rc = flux_attn_prefill(plan, layer, req, q_dev, k, v, q_start, Nq, out_dev, stream);
    if (!rc) rc = check_cuda(cudaMemcpyAsync(out_host, out_dev, qb, cudaMemcpyDeviceToHost, st), "out download");
    return rc;
}

int flux_plan_status(flux_plan *plan, uint32_t *status_bits, void *stream)
{
    int rc = need_plan(plan, true);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    uint32_t bits = 0;
    void *d = (char *)plan->ws + plan->lay.status;
    rc = check_cuda(cudaMemcpyAsync(&bits, d, sizeof bits, cudaMemcpyDeviceToHost, st), "status read");
    if (!rc) rc = check_cuda(cudaMemsetAsync(d, 0, sizeof bits, st), "status clear");
    if (!rc) rc = check_cuda(cudaStreamSynchronize(st), "stream synchronize");
    if (rc) return rc;
    if (bits & FLUX_STATUS_WAIT_EXPIRED) {   // a kernel left early: its arrival counters are not back at zero
        // the router's counters and launch number, and with them the tagged activations (an old tag must not match)
        rc = check_cuda(cudaMemsetAsync((char *)plan->ws + plan->lay.router, 0,
                                        plan->lay.router_sync + 8 * sizeof(uint32_t) - plan->lay.router, st), "counter clear");
        if (!rc) rc = check_cuda(cudaMemsetAsync((char *)plan->ws + plan->lay.tickets, 0,
                                                 plan->lay.push_ticket + 8 * sizeof(uint32_t) - plan->lay.tickets, st), "counter clear");
        if (!rc) rc = check_cuda(cudaStreamSynchronize(st), "stream synchronize");
        if (rc) return rc;
    }
    if (status_bits) *status_bits = bits;
    if (bits & FLUX_STATUS_WAIT_EXPIRED)
        return fail(FLUX_E_DEVICE_TIMEOUT, "a device-side wait expired (status 0x%x)", bits);
    if (bits) return fail(FLUX_E_DEVICE_FLAG, "device-side input check failed (status 0x%x)", bits);
    return FLUX_OK;
}

int flux_debug_dispatch(flux_plan *plan, int32_t *records_out, int32_t max_records,
                        int32_t *n_records_out, void *stream)
{
    int rc = need_plan(plan, true);
    if (rc) return rc;
    if (!records_out || !n_records_out || max_records < 0)
        return fail(FLUX_E_INVALID_ARG, "bad output arguments");
    cudaStream_t st = (cudaStream_t)stream;
    int n = plan->debug_records < max_records ? plan->debug_records : max_records;
    if (n > 0) {
        rc = check_cuda(cudaMemcpyAsync(records_out, (char *)plan->ws + plan->lay.debug,
                                        (size_t)n * 8 * sizeof(int32_t), cudaMemcpyDeviceToHost, st),
                        "dispatch record read");
        if (rc) return rc;
    }
    rc = check_cuda(cudaStreamSynchronize(st), "stream synchronize");
    if (rc) return rc;
    *n_records_out = n;
    return FLUX_OK;
}

int flux_profile_enable(flux_plan *plan, int32_t max_records)
{
    int rc = need_plan(plan, false);
    if (rc) return rc;
    if (max_records < 0 || max_records > (1 << 20))
        return fail(FLUX_E_INVALID_ARG, "max_records outside [0, 2^20]");
    prof_free(plan);
    if (max_records == 0) return FLUX_OK;
    plan->prof_ev = (cudaEvent_t *)calloc(2 * (size_t)max_records, sizeof(cudaEvent_t));
    plan->prof_kind = (int8_t *)calloc((size_t)max_records, 1);
    if (!plan->prof_ev || !plan->prof_kind) {
        free(plan->prof_ev);
        free(plan->prof_kind);
        plan->prof_ev = nullptr;
        plan->prof_kind = nullptr;
        return fail(FLUX_E_INVALID_ARG, "out of host memory");
    }
    for (int i = 0; i < 2 * max_records; ++i) {
        rc = check_cuda(cudaEventCreate(&plan->prof_ev[i]), "cudaEventCreate");
        if (rc) {
            plan->prof_cap = (i + 1) / 2;
            prof_free(plan);
            return rc;
        }
    }
    plan->prof_cap = max_records;
    plan->prof_n = 0;
    return FLUX_OK;
}

int flux_profile_read(flux_plan *plan, int32_t kind, double *total_ms, int64_t *launches, void *stream)
{
    int rc = need_plan(plan, false);
    if (rc) return rc;
    if (!total_ms || !launches) return fail(FLUX_E_INVALID_ARG, "NULL output pointer");
    rc = check_cuda(cudaStreamSynchronize((cudaStream_t)stream), "stream synchronize");
    if (rc) return rc;
    double sum = 0.0;
    int64_t cnt = 0;
    for (int i = 0; i < plan->prof_n; ++i) {
        if (plan->prof_kind[i] != kind) continue;
        float ms = 0.f;
        rc = check_cuda(cudaEventElapsedTime(&ms, plan->prof_ev[2 * i], plan->prof_ev[2 * i + 1]),
                        "cudaEventElapsedTime");
        if (rc) return rc;
        sum += ms;
        ++cnt;
    }
    plan->prof_n = 0;
    *total_ms = sum;
    *launches = cnt;
    return FLUX_OK;
}

int64_t flux_launch_count(const flux_plan *plan) { return plan ? plan->launches : 0; }

}  // extern "C"
