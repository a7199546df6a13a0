/*
 * CPU oracle for the WindowKV prefill-time window selection path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of the
 * paper's definitions that the CUDA library is checked against.  Nothing in
 * the product path may call it; it shares no code, header, table or helper
 * with the CUDA sources.  Floating-point work is done in double precision on
 * inputs widened exactly from fp32 / bf16.
 *
 * Passages followed (paper section 2.2.1 and 2.2.2):
 *   observation / review split ........ first paragraph of "Task-Adaptive Window Selection"
 *   Eq. 1  A = softmax(Q K^T / sqrt(d_k))
 *   Eq. 2  t_j = sum over observation rows i of A_ij, j in the review context
 *   Eq. 3  review windows of omega consecutive tokens, ceil((n - alpha)/omega) of them
 *   Eq. 4  s_k = sum(Top-p(W_k)) / min(p, omega)
 *   budget sentence after Eq. 4 ....... keep the highest-scoring windows that fit the budget
 *   intra-group sharing ............... the leader's indices are reused by every layer of the group
 *
 * Readings taken where the paper is silent (each is a convention, stated in
 * the design notes): half-open index ranges in Eq. 2; the softmax row is the
 * model's causal row (keys 0..i, observation keys included in the
 * normaliser); scores are summed over the G query heads that share a KV head;
 * a ragged last window keeps its real size and divides by min(p, size); the
 * budget b counts the alpha observation rows, k = floor((b - alpha)/omega);
 * ties go to the lower window index; retained rows are emitted in ascending
 * position, review rows first, observation rows last.
 *
 * Parity pins: every function below is pinned by tests that do not use this
 * file's own arithmetic (closed forms, row-sum invariant, a library softmax,
 * library pooling, exhaustive subset enumeration, hand-worked rational
 * examples).  The paper prints no worked numeric example of Eq. 1-4, so the
 * *readings* listed above are "parity unpinned" by the paper itself.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define WKVO_F32 0
#define WKVO_BF16 1

static double load_elem(const void *base, int dtype, int64_t idx)
{
    if (dtype == WKVO_F32)
        return (double)((const float *)base)[idx];
    uint32_t u = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static int elem_size(int dtype) { return dtype == WKVO_F32 ? 4 : 2; }

int wkvo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- integer helpers (budget sentence after Eq. 4; Eq. 3) ---------------- */

/* number of review windows, Eq. 3 */
int64_t wkvo_num_windows(int64_t n, int64_t alpha, int64_t omega)
{
    if (n <= alpha)
        return 0;
    return (n - alpha + omega - 1) / omega;
}

/* number of windows retained under a per-layer budget of b tokens that
 * includes the observation window */
int64_t wkvo_num_selected(int64_t n, int64_t alpha, int64_t omega, int64_t b)
{
    int64_t kw = wkvo_num_windows(n, alpha, omega);
    int64_t k = b > alpha ? (b - alpha) / omega : 0;
    return k < kw ? k : kw;
}

/* ---- Eq. 1-2: token scores of one (sequence, KV head) unit --------------- */
/*
 * q : first query head of the KV head's group; element (g, i, c) at
 *     q[g*q_stride_h + i*q_stride_t + c], i = 0..alpha-1 are the last alpha
 *     positions n-alpha .. n-1.
 * k : keys of the unit; element (j, c) at k[j*k_stride_t + c], j = 0..n-1.
 * t_out      [n - alpha]  token scores (Eq. 2), double
 * obs_mass   optional: attention mass that the observation rows put on the
 *            observation keys themselves (for the row-sum invariant)
 * lse_out    optional [G*alpha]: log of the softmax normaliser, natural log
 */
void wkvo_token_scores_unit(int dtype, const void *q, int64_t q_stride_h, int64_t q_stride_t,
                            const void *k, int64_t k_stride_t,
                            int64_t n, int64_t alpha, int64_t G, int64_t d,
                            double *t_out, double *obs_mass, double *lse_out)
{
    int64_t n_r = n - alpha;
    if (obs_mass)
        *obs_mass = 0.0;
    if (n_r <= 0)
        return;
    for (int64_t j = 0; j < n_r; ++j)
        t_out[j] = 0.0;

    double *kd = (double *)malloc(sizeof(double) * (size_t)n * (size_t)d);
    double *qd = (double *)malloc(sizeof(double) * (size_t)d);
    double *s = (double *)malloc(sizeof(double) * (size_t)n);
    for (int64_t j = 0; j < n; ++j)
        for (int64_t c = 0; c < d; ++c)
            kd[j * d + c] = load_elem(k, dtype, j * k_stride_t + c);

    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    for (int64_t g = 0; g < G; ++g) {
        for (int64_t i = 0; i < alpha; ++i) {
            int64_t pos = n_r + i;              /* absolute position of this query */
            for (int64_t c = 0; c < d; ++c)
                qd[c] = load_elem(q, dtype, g * q_stride_h + i * q_stride_t + c);
            /* Eq. 1, one row: logits over the keys this position may attend to */
            double m = -INFINITY;
            for (int64_t j = 0; j <= pos; ++j) {
                double acc = 0.0;
                const double *kj = kd + j * d;
                for (int64_t c = 0; c < d; ++c)
                    acc += qd[c] * kj[c];
                s[j] = acc * inv_sqrt_d;
                if (s[j] > m)
                    m = s[j];
            }
            double z = 0.0;
            for (int64_t j = 0; j <= pos; ++j) {
                s[j] = exp(s[j] - m);
                z += s[j];
            }
            /* Eq. 2: add this row's attention to every review token */
            for (int64_t j = 0; j < n_r; ++j)
                t_out[j] += s[j] / z;
            if (obs_mass)
                for (int64_t j = n_r; j <= pos; ++j)
                    *obs_mass += s[j] / z;
            if (lse_out)
                lse_out[g * alpha + i] = m + log(z);
        }
    }
    free(s);
    free(qd);
    free(kd);
}

/* ---- Eq. 3-4: window scores ---------------------------------------------- */
static int cmp_desc_double(const void *a, const void *b)
{
    double x = *(const double *)a, y = *(const double *)b;
    return (x < y) - (x > y);
}

/* t [n_r] -> s [ceil(n_r/omega)] (double) ; p is the Top-p count (p = omega
 * for the localization task) */
void wkvo_window_scores(const double *t, int64_t n_r, int64_t omega, int64_t p, double *s_out)
{
    int64_t kw = (n_r + omega - 1) / omega;
    double *buf = (double *)malloc(sizeof(double) * (size_t)omega);
    for (int64_t w = 0; w < kw; ++w) {
        int64_t lo = w * omega;
        int64_t hi = lo + omega < n_r ? lo + omega : n_r;
        int64_t size = hi - lo;
        for (int64_t x = 0; x < size; ++x)
            buf[x] = t[lo + x];
        qsort(buf, (size_t)size, sizeof(double), cmp_desc_double);
        int64_t pk = p < size ? p : size;
        double acc = 0.0;
        for (int64_t x = 0; x < pk; ++x)
            acc += buf[x];
        s_out[w] = acc / (double)pk;
    }
    free(buf);
}

/* ---- budgeted selection --------------------------------------------------- */
typedef struct {
    float score;
    int32_t index;
} wkvo_cand;

static int cmp_cand(const void *a, const void *b)
{
    const wkvo_cand *x = (const wkvo_cand *)a, *y = (const wkvo_cand *)b;
    if (x->score > y->score)
        return -1;
    if (x->score < y->score)
        return 1;
    return (x->index > y->index) - (x->index < y->index);
}

static int cmp_i32(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/* the k highest fp32 scores, ties to the lower index; indices ascending */
void wkvo_select_topk(const float *scores, int64_t kw, int64_t k, int32_t *idx_out)
{
    if (k <= 0)
        return;
    wkvo_cand *c = (wkvo_cand *)malloc(sizeof(wkvo_cand) * (size_t)kw);
    for (int64_t w = 0; w < kw; ++w) {
        c[w].score = scores[w];
        c[w].index = (int32_t)w;
    }
    qsort(c, (size_t)kw, sizeof(wkvo_cand), cmp_cand);
    for (int64_t x = 0; x < k; ++x)
        idx_out[x] = c[x].index;
    qsort(idx_out, (size_t)k, sizeof(int32_t), cmp_i32);
    free(c);
}

/* ---- gather of one unit of one layer -------------------------------------- */
/* copies rows idx[x]*omega .. (clipped at n - alpha) then rows n-alpha..n-1.
 * returns the number of rows written. src/dst rows are d elements, row
 * strides in elements. */
int64_t wkvo_gather_unit(int dtype, const void *src, int64_t src_stride_t,
                         void *dst, int64_t dst_stride_t,
                         int64_t n, int64_t alpha, int64_t omega, int64_t d,
                         const int32_t *idx, int64_t k)
{
    int es = elem_size(dtype);
    int64_t n_r = n > alpha ? n - alpha : 0;
    int64_t r = 0;
    for (int64_t x = 0; x < k; ++x) {
        int64_t lo = (int64_t)idx[x] * omega;
        int64_t hi = lo + omega < n_r ? lo + omega : n_r;
        for (int64_t j = lo; j < hi; ++j, ++r)
            memcpy((char *)dst + r * dst_stride_t * es, (const char *)src + j * src_stride_t * es,
                   (size_t)(d * es));
    }
    for (int64_t j = n_r; j < n; ++j, ++r)
        memcpy((char *)dst + r * dst_stride_t * es, (const char *)src + j * src_stride_t * es,
               (size_t)(d * es));
    return r;
}

/* ---- whole leader: scores + selection for every unit of a batch ----------- */
/*
 * Layout convention (element strides, d contiguous):
 *   K element (b, h, j, c) at  k[seq_off(b)*stride_t + b*stride_b + h*stride_h + j*stride_t + c]
 *   where seq_off(b) = cu_seqlens[b] for the packed layout (stride_b = 0) and 0 otherwise.
 *   Q_obs element (b, hq, i, c) at q[b*q_stride_b + hq*q_stride_h + i*q_stride_t + c].
 * Outputs, all [B, H_kv, ...] row-major with the given leading sizes:
 *   win_scores_d [B,H_kv,kw_max] double (optional), win_scores [B,H_kv,kw_max] fp32,
 *   token_scores [B,H_kv,nr_max] double (optional),
 *   win_idx [B,H_kv,k_max] int32 ascending, padded with -1, kept_len [B,H_kv] int32.
 * unit_mask (optional, [B*H_kv]): units with a zero entry are skipped (sampled parity).
 */
void wkvo_select_leader(int dtype, const void *q, const void *k,
                        int64_t B, int64_t Hq, int64_t Hkv, int64_t d,
                        int64_t alpha, int64_t omega, int64_t p,
                        int64_t max_seqlen, const int32_t *cu_seqlens, const int32_t *budgets,
                        int64_t stride_b, int64_t stride_h, int64_t stride_t,
                        int64_t q_stride_b, int64_t q_stride_h, int64_t q_stride_t,
                        int64_t kw_max, int64_t nr_max, int64_t k_max,
                        double *win_scores_d, float *win_scores, double *token_scores,
                        int32_t *win_idx, int32_t *kept_len, const uint8_t *unit_mask)
{
    int64_t G = Hq / Hkv;
    int es = elem_size(dtype);
    int64_t units = B * Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t u = 0; u < units; ++u) {
        if (unit_mask && !unit_mask[u])
            continue;
        int64_t b = u / Hkv, h = u % Hkv;
        int64_t n = cu_seqlens ? (int64_t)(cu_seqlens[b + 1] - cu_seqlens[b]) : max_seqlen;
        int64_t off = cu_seqlens ? (int64_t)cu_seqlens[b] : 0;
        int64_t n_r = n > alpha ? n - alpha : 0;
        int64_t kw = wkvo_num_windows(n, alpha, omega);
        int64_t ksel = wkvo_num_selected(n, alpha, omega, budgets[b]);
        int32_t *idx = win_idx + u * k_max;
        for (int64_t x = 0; x < k_max; ++x)
            idx[x] = -1;
        int64_t kept = n < alpha ? n : alpha;
        if (kw > 0) {
            const char *ku = (const char *)k + (off * stride_t + b * stride_b + h * stride_h) * es;
            const char *qu = (const char *)q + (b * q_stride_b + h * G * q_stride_h) * es;
            double *t = (double *)malloc(sizeof(double) * (size_t)n_r);
            double *sd = (double *)malloc(sizeof(double) * (size_t)kw);
            wkvo_token_scores_unit(dtype, qu, q_stride_h, q_stride_t, ku, stride_t, n, alpha, G, d,
                                   t, NULL, NULL);
            wkvo_window_scores(t, n_r, omega, p, sd);
            float *sf = win_scores + u * kw_max;
            for (int64_t w = 0; w < kw; ++w)
                sf[w] = (float)sd[w];
            if (win_scores_d)
                memcpy(win_scores_d + u * kw_max, sd, sizeof(double) * (size_t)kw);
            if (token_scores)
                memcpy(token_scores + u * nr_max, t, sizeof(double) * (size_t)n_r);
            wkvo_select_topk(sf, kw, ksel, idx);
            for (int64_t x = 0; x < ksel; ++x) {
                int64_t lo = (int64_t)idx[x] * omega;
                int64_t hi = lo + omega < n_r ? lo + omega : n_r;
                kept += hi - lo;
            }
            free(sd);
            free(t);
        }
        kept_len[u] = (int32_t)kept;
    }
}

/* ---- gather of one layer for every unit ------------------------------------ */
/* dst is dense [B, H_kv, keep_max, d] when cu_seqlens_out == NULL, else packed
 * [T_out, H_kv, d] with sequence b starting at row cu_seqlens_out[b]. */
void wkvo_gather_layer(int dtype, const void *src, void *dst,
                       int64_t B, int64_t Hkv, int64_t d, int64_t alpha, int64_t omega,
                       int64_t max_seqlen, const int32_t *cu_seqlens,
                       int64_t stride_b, int64_t stride_h, int64_t stride_t,
                       const int32_t *win_idx, int64_t k_max, const int32_t *budgets,
                       int64_t keep_max, const int32_t *cu_seqlens_out)
{
    int es = elem_size(dtype);
    int64_t units = B * Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t u = 0; u < units; ++u) {
        int64_t b = u / Hkv, h = u % Hkv;
        int64_t n = cu_seqlens ? (int64_t)(cu_seqlens[b + 1] - cu_seqlens[b]) : max_seqlen;
        int64_t off = cu_seqlens ? (int64_t)cu_seqlens[b] : 0;
        int64_t ksel = wkvo_num_selected(n, alpha, omega, budgets[b]);
        const char *su = (const char *)src + (off * stride_t + b * stride_b + h * stride_h) * es;
        char *du;
        int64_t dst_stride_t;
        if (cu_seqlens_out) {
            du = (char *)dst + ((int64_t)cu_seqlens_out[b] * Hkv * d + h * d) * es;
            dst_stride_t = Hkv * d;
        } else {
            du = (char *)dst + ((b * Hkv + h) * keep_max * d) * es;
            dst_stride_t = d;
        }
        wkvo_gather_unit(dtype, su, stride_t, du, dst_stride_t, n, alpha, omega, d,
                         win_idx + u * k_max, ksel);
    }
}
