/*
 * flux_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, fp64 CPU statement of what routed hybrid attention computes
 * (Flux Attention: a layer runs Full Attention or Sparse Attention, chosen by
 * a cached per-request hard routing bit).  Only tests, the smoke check and the
 * benchmark's cpu_baseline / reference legs may call it.  It shares no source,
 * header, table or helper with the CUDA library.
 *
 * Everything here is the definition written out:
 *   - Full Attention, Eq. 1:    O_r = Softmax(Q K^T) V        (causal decoder)
 *   - Sparse Attention, Eq. 2:  O_s = Softmax(Q K~^T) V~      with (K~, V~) the
 *     streaming subset: the first S positions (attention sink) and the last W
 *     positions up to and including the query's own position (local window),
 *     Sec. 4.1 "Streaming Sparse Attention" and the Sparsity Config of Table 3.
 *   - Hard routing, Sec. 3.1 "Deterministic Inference via Hard Routing":
 *     r_hard = argmax(pi_FA, pi_SA);  r_hard == 0 runs SA.
 *   - Model Sparsity Ratio, Eq. 3: fraction of (layer, head) slots in SA mode.
 *   - Sparse-decode KV retention, Sec. 3.3: an SA layer keeps only the rows
 *     its kernel needs; an FA layer keeps every row.
 *
 * No blocking, no online softmax, no reordering: each output row is computed
 * from an explicit sorted list of kept key indices, scores first, then max,
 * then exponentials, then the normalised weighted sum.
 *
 * Inputs are bf16 bit patterns (uint16_t), upcast exactly to double; the paper
 * runs in bfloat16 (Appendix C.3), so bf16 is the input precision and fp64 the
 * arithmetic.  Layouts: Q, O [rows][Hq][D]; K, V [tokens][Hkv][D] with an
 * explicit token stride in elements.  GQA: query head h reads KV head
 * h / (Hq / Hkv).  The softmax scale is a parameter (Eq. 1 omits it).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define FLUX_ORACLE_FA 1
#define FLUX_ORACLE_SA 0

static double bf16_bits_to_f64(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ---- kept index sets (Eq. 1 / Eq. 2 with the sink + window subset) --------
 * mode FA: { j : 0 <= j <= i }
 * mode SA: { j : 0 <= j <= i  and  ( j < S  or  j > i - W ) }
 * Writes the sorted list into idx (room for i+1 entries) and returns its size.
 * idx may be NULL to count only. */
int64_t flux_oracle_kept(int mode, int64_t i, int64_t S, int64_t W, int64_t *idx)
{
    int64_t cnt = 0;
    for (int64_t j = 0; j <= i; ++j) {
        int keep;
        if (mode == FLUX_ORACLE_FA)
            keep = 1;
        else
            keep = (j < S) || (j > i - W);
        if (keep) {
            if (idx) idx[cnt] = j;
            ++cnt;
        }
    }
    return cnt;
}

/* ---- one output row: softmax over an explicit index list -------------------
 * q: [D] bf16 bits.  K, V: base of one KV head, token j at K + j*tok_stride.
 * o: [D] fp64.  p (optional): [n_idx] normalised probabilities.
 * m_out / l_out (optional): row maximum of the scaled scores and the sum of
 * exp(score - max), i.e. the log-sum-exp pieces a split evaluation would merge.
 */
void flux_oracle_attend(const uint16_t *q, const uint16_t *K, const uint16_t *V,
                        int64_t tok_stride, const int64_t *idx, int64_t n_idx,
                        int D, double scale, double *o, double *p,
                        double *m_out, double *l_out)
{
    double *s = (double *)malloc(sizeof(double) * (size_t)(n_idx > 0 ? n_idx : 1));
    double m = -INFINITY;
    for (int64_t t = 0; t < n_idx; ++t) {
        const uint16_t *k = K + idx[t] * tok_stride;
        double acc = 0.0;
        for (int d = 0; d < D; ++d)
            acc += bf16_bits_to_f64(q[d]) * bf16_bits_to_f64(k[d]);
        s[t] = scale * acc;
        if (s[t] > m) m = s[t];
    }
    double l = 0.0;
    for (int64_t t = 0; t < n_idx; ++t) {
        s[t] = exp(s[t] - m);
        l += s[t];
    }
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    for (int64_t t = 0; t < n_idx; ++t) {
        const uint16_t *v = V + idx[t] * tok_stride;
        double w = s[t] / l;
        if (p) p[t] = w;
        for (int d = 0; d < D; ++d)
            o[d] += w * bf16_bits_to_f64(v[d]);
    }
    if (m_out) *m_out = m;
    if (l_out) *l_out = l;
    free(s);
}

/* ---- prefill of one layer for one request ----------------------------------
 * Query rows sit at absolute positions q_start .. q_start+Nq-1; the KV arrays
 * hold positions 0 .. q_start+Nq-1 (chunked prefill, Appendix D.3 "chunk
 * size": earlier chunks' keys are already there).  mode: 1 = FA, 0 = SA. */
void flux_oracle_prefill(int mode, const uint16_t *Q, const uint16_t *K,
                         const uint16_t *V, int64_t kv_tok_stride,
                         int64_t q_start, int64_t Nq, int Hq, int Hkv, int D,
                         int64_t S, int64_t W, double scale, double *O)
{
    int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 4)
    for (int64_t r = 0; r < Nq; ++r) {
        for (int h = 0; h < Hq; ++h) {
            int64_t i = q_start + r;
            int64_t *idx = (int64_t *)malloc(sizeof(int64_t) * (size_t)(i + 1));
            int64_t n_idx = flux_oracle_kept(mode, i, S, W, idx);
            int g = h / G;
            flux_oracle_attend(Q + (r * Hq + h) * (int64_t)D, K + (int64_t)g * D,
                               V + (int64_t)g * D, kv_tok_stride, idx, n_idx, D,
                               scale, O + (r * Hq + h) * (int64_t)D, NULL, NULL,
                               NULL);
            free(idx);
        }
    }
}

/* ---- selected prefill rows (for sampled checks at sizes too big to sweep) --
 * rows[t] is an absolute query position, heads[t] a query head; Q is indexed
 * by (rows[t] - q_start).  O: [n_rows][D]. */
void flux_oracle_prefill_rows(int mode, const uint16_t *Q, const uint16_t *K,
                              const uint16_t *V, int64_t kv_tok_stride,
                              int64_t q_start, const int64_t *rows,
                              const int32_t *heads, int64_t n_rows, int Hq,
                              int Hkv, int D, int64_t S, int64_t W,
                              double scale, double *O)
{
    int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t t = 0; t < n_rows; ++t) {
        int64_t i = rows[t];
        int h = heads[t];
        int64_t *idx = (int64_t *)malloc(sizeof(int64_t) * (size_t)(i + 1));
        int64_t n_idx = flux_oracle_kept(mode, i, S, W, idx);
        int g = h / G;
        flux_oracle_attend(Q + ((i - q_start) * Hq + h) * (int64_t)D,
                           K + (int64_t)g * D, V + (int64_t)g * D, kv_tok_stride,
                           idx, n_idx, D, scale, O + t * (int64_t)D, NULL, NULL,
                           NULL);
        free(idx);
    }
}

/* ---- block-granular sparse patterns ----------------------------------------
 * The sparse kernels the paper runs select keys in blocks (Appendix D.3: the
 * block size, 64, is the granularity at which keys are kept or dropped; Sec. 4.1 lists block
 * patterns -- streaming, XAttention's selected blocks -- as the sparse modes).
 * A block mask bm[qb][kb] (row-major, n_kb entries per row) says whether query
 * block qb (positions [qb*B, (qb+1)*B)) attends to key block kb; inside a kept
 * block causality still holds:
 *     kept(i) = { j : 0 <= j <= i  and  bm[i / B][j / B] != 0 }
 * B = 1 makes bm an arbitrary token-level mask.  Writes the sorted list into
 * idx (room for i+1 entries, may be NULL) and returns its size. */
int64_t flux_oracle_kept_blocks(int64_t i, int64_t B, const uint8_t *bm,
                                int64_t n_kb, int64_t *idx)
{
    int64_t cnt = 0;
    const uint8_t *row = bm + (i / B) * n_kb;
    for (int64_t j = 0; j <= i; ++j) {
        if (row[j / B] != 0) {
            if (idx) idx[cnt] = j;
            ++cnt;
        }
    }
    return cnt;
}

/* Prefill rows under a block mask (Eq. 2 with the condensed subset given by the
 * mask).  rows / heads as in flux_oracle_prefill_rows; rows == NULL evaluates
 * every (row, head) of the chunk in order, O then [Nq][Hq][D].  A query whose
 * kept set is empty gets a zero row. */
void flux_oracle_prefill_blocks(const uint16_t *Q, const uint16_t *K,
                                const uint16_t *V, int64_t kv_tok_stride,
                                int64_t q_start, int64_t Nq, const int64_t *rows,
                                const int32_t *heads, int64_t n_rows, int Hq,
                                int Hkv, int D, int64_t B, const uint8_t *bm,
                                int64_t n_kb, double scale, double *O)
{
    int G = Hq / Hkv;
    int64_t total = rows ? n_rows : Nq * Hq;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t t = 0; t < total; ++t) {
        int64_t i = rows ? rows[t] : q_start + t / Hq;
        int h = rows ? heads[t] : (int)(t % Hq);
        int64_t *idx = (int64_t *)malloc(sizeof(int64_t) * (size_t)(i + 1));
        int64_t n_idx = flux_oracle_kept_blocks(i, B, bm, n_kb, idx);
        double *o = O + t * (int64_t)D;
        if (n_idx == 0) {
            for (int d = 0; d < D; ++d) o[d] = 0.0;
        } else {
            int g = h / G;
            flux_oracle_attend(Q + ((i - q_start) * Hq + h) * (int64_t)D,
                               K + (int64_t)g * D, V + (int64_t)g * D,
                               kv_tok_stride, idx, n_idx, D, scale, o, NULL,
                               NULL, NULL);
        }
        free(idx);
    }
}

/* ---- one decode step of one layer for one request --------------------------
 * The new token's K, V were appended first, so the cache holds positions
 * 0 .. n-1 and the query sits at position n-1 (Sec. 3.3).  q, o: [Hq][D].
 * heads (optional, n_heads entries) restricts the evaluation to some query
 * heads; o is then [n_heads][D]. */
void flux_oracle_decode(int mode, const uint16_t *q, const uint16_t *K,
                        const uint16_t *V, int64_t kv_tok_stride, int64_t n,
                        int Hq, int Hkv, int D, int64_t S, int64_t W,
                        double scale, const int32_t *heads, int n_heads,
                        double *o)
{
    int G = Hq / Hkv;
    int cnt = heads ? n_heads : Hq;
    int64_t *idx = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
    int64_t n_idx = flux_oracle_kept(mode, n - 1, S, W, idx);
#pragma omp parallel for schedule(dynamic, 1)
    for (int t = 0; t < cnt; ++t) {
        int h = heads ? heads[t] : t;
        int g = h / G;
        flux_oracle_attend(q + (int64_t)h * D, K + (int64_t)g * D,
                           V + (int64_t)g * D, kv_tok_stride, idx, n_idx, D,
                           scale, o + (int64_t)t * D, NULL, NULL, NULL);
    }
    free(idx);
}

/* ---- hard routing (Sec. 3.1): mask = argmax over (pi_FA, pi_SA) -------------
 * logits: [B][L][2], FA logit first.  mask[b][l] = 1 (FA) or 0 (SA).  A tie
 * goes to FA.  Returns the number of NaN logits met (their mask byte is 0xFF).
 */
int64_t flux_oracle_route(const float *logits, int64_t B, int64_t L,
                          uint8_t *mask)
{
    int64_t bad = 0;
    for (int64_t t = 0; t < B * L; ++t) {
        float fa = logits[2 * t], sa = logits[2 * t + 1];
        if (isnan(fa) || isnan(sa)) {
            mask[t] = 0xFF;
            ++bad;
        } else {
            mask[t] = (fa >= sa) ? 1 : 0;
        }
    }
    return bad;
}

/* ---- Model Sparsity Ratio (Eq. 3) -------------------------------------------
 * All H heads of a layer share the layer's mode, so the double sum over
 * (layer, head) slots reduces to the fraction of SA layers; written out as in
 * Eq. 3 anyway. */
double flux_oracle_msr(const uint8_t *mask, int64_t L, int64_t H)
{
    int64_t sa = 0;
    for (int64_t l = 0; l < L; ++l)
        for (int64_t h = 0; h < H; ++h)
            sa += (mask[l] == 0);
    return (double)sa / (double)(H * L);
}

/* ---- sparse-decode KV retention (Sec. 3.3) ---------------------------------
 * Positions an SA layer must still hold when the context has n tokens: the
 * kept set of the newest query (position n-1).  Later queries never need an
 * evicted row again because the window only moves forward. */
int64_t flux_oracle_retained(int64_t n, int64_t S, int64_t W, int64_t *idx)
{
    return flux_oracle_kept(FLUX_ORACLE_SA, n - 1, S, W, idx);
}

/* Slot of position j in a compact SA cache of S + W rows: sink rows stay in
 * place, the rest go round a ring of W rows.  (A storage rule of this build,
 * not of the paper; the oracle states it independently so that the library's
 * ring writes can be checked row by row.) */
int64_t flux_oracle_compact_slot(int64_t j, int64_t S, int64_t W)
{
    if (j < S) return j;
    return S + ((j - S) % W);
}

/* ---- merging two partial softmax evaluations --------------------------------
 * Attention over a disjoint union I1 + I2 from the pieces (m, l, o) of each
 * part, where o is the *normalised* output of the part, m its maximum score
 * and l its sum of exp(score - m).  Derived from Eq. 1 by splitting the sums.
 */
void flux_oracle_merge(int D, double m1, double l1, const double *o1, double m2,
                       double l2, const double *o2, double *m, double *l,
                       double *o)
{
    double mm = m1 > m2 ? m1 : m2;
    double a1 = l1 * exp(m1 - mm), a2 = l2 * exp(m2 - mm);
    for (int d = 0; d < D; ++d)
        o[d] = (a1 * o1[d] + a2 * o2[d]) / (a1 + a2);
    *m = mm;
    *l = a1 + a2;
}
