// Host side of the C ABI: argument validation, shape resolution, workspace
// carve-up and kernel sequencing.  No device memory is allocated here.
#include "wkv_internal.cuh"

#include <atomic>
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

namespace wkv {

static thread_local char g_detail[512] = "";
static std::atomic<uint64_t> g_launches{0};

void set_error_detail(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_detail, sizeof g_detail, fmt, ap);
    va_end(ap);
}

void count_launches(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

size_t score_simt_smem_bytes(const KShape &ks, int r_pad);

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

Workspace plan_workspace(const KShape &ks)
{
    Workspace w;
    const size_t units = (size_t)ks.batch * ks.hkv;
    w.r_pad = (ks.R + 63) / 64 * 64;
    w.n_stat_chunks = (ks.max_seqlen + kStatChunk - 1) / kStatChunk;
    const int tc_chunks = tc_plan((int)units, ks.max_seqlen, ks.d).chunks_per_unit;
    if (tc_chunks > w.n_stat_chunks) w.n_stat_chunks = tc_chunks;
    const int pipe_chunks = pipe_plan((int)units, ks.max_seqlen, ks.d).chunks_per_unit;
    if (pipe_chunks > w.n_stat_chunks) w.n_stat_chunks = pipe_chunks;
    size_t off = 0;
    w.status_off = off;
    off = 64;
    w.sync_off = off;
    off = align_up(off + (kSyncTickets + kSyncWordsPerUnit * (size_t)units) * sizeof(int), 256);
    w.pstats_off = off;
    off = align_up(off + (ks.R <= 128 ? units * w.n_stat_chunks * 128 * sizeof(unsigned long long) : 0), 256);
    w.stats_off = off;
    off = align_up(off + units * w.n_stat_chunks * w.r_pad * sizeof(float2), 256);
    w.lse_off = off;
    off = align_up(off + units * w.r_pad * sizeof(float), 256);
    w.scores_off = off;
    off = align_up(off + units * (size_t)ks.kw_max * sizeof(float), 256);
    w.total = off;
    return w;
}

static int elem_bytes(int dtype) { return dtype == WKV_F32 ? 4 : 2; }

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Validates the shape and fills the kernel-side copy.  `seqlens` are read from the host arrays.
int resolve(const wkv_shape *s, KShape &ks)
{
    if (!s) {
        set_error_detail("shape is NULL");
        return WKV_ERR_NULL;
    }
    if (s->struct_size != sizeof(wkv_shape)) {
        set_error_detail("struct_size %u != %zu", s->struct_size, sizeof(wkv_shape));
        return WKV_ERR_SHAPE;
    }
    if (s->dtype != WKV_F32 && s->dtype != WKV_BF16) {
        set_error_detail("dtype %d unknown", s->dtype);
        return WKV_ERR_DTYPE;
    }
    if (s->batch < 1 || s->n_q_heads < 1 || s->n_kv_heads < 1 || s->head_dim < 1 || s->l_obs < 1 ||
        s->window < 1 || s->max_seqlen < 1 || s->top_p < 0) {
        set_error_detail("non-positive size (batch %d, heads %d/%d, d %d, alpha %d, omega %d, N %d, p %d)",
                         s->batch, s->n_q_heads, s->n_kv_heads, s->head_dim, s->l_obs, s->window,
                         s->max_seqlen, s->top_p);
        return WKV_ERR_SHAPE;
    }
    if (s->n_q_heads % s->n_kv_heads) {
        set_error_detail("n_q_heads %d not a multiple of n_kv_heads %d", s->n_q_heads, s->n_kv_heads);
        return WKV_ERR_SHAPE;
    }
    if (s->task != WKV_TASK_LOCALIZATION && s->task != WKV_TASK_AGGREGATION) {
        set_error_detail("task %d unknown", s->task);
        return WKV_ERR_SHAPE;
    }
    if (s->score_impl < WKV_SCORE_AUTO || s->score_impl > WKV_SCORE_TCGEN05_PIPELINED || s->reserved != 0) {
        set_error_detail("score_impl %d / reserved %d invalid", s->score_impl, s->reserved);
        return WKV_ERR_SHAPE;
    }
    const int eb = elem_bytes(s->dtype);
    if ((s->head_dim * eb) % 16) {
        set_error_detail("head_dim %d: a row must be a multiple of 16 bytes", s->head_dim);
        return WKV_ERR_ALIGN;
    }
    const int64_t strides[6] = {s->stride_b, s->stride_h, s->stride_t,
                                s->q_stride_b, s->q_stride_h, s->q_stride_t};
    for (int i = 0; i < 6; ++i) {
        if (strides[i] < 0 || (strides[i] * eb) % 16) {
            set_error_detail("stride #%d = %lld is negative or not 16-byte aligned", i, (long long)strides[i]);
            return WKV_ERR_ALIGN;
        }
    }
    if (s->stride_t < s->head_dim || s->q_stride_t < s->head_dim) {
        set_error_detail("token stride smaller than head_dim");
        return WKV_ERR_SHAPE;
    }
    if ((s->cu_seqlens_host == nullptr) != (s->cu_seqlens_dev == nullptr) ||
        (s->budgets_host == nullptr) != (s->budgets_dev == nullptr)) {
        set_error_detail("host and device copies of cu_seqlens / budgets must be given together");
        return WKV_ERR_NULL;
    }
    long long total = 0;
    int kw_max = 1, k_max = 1, nr_max = 1;
    for (int b = 0; b < s->batch; ++b) {
        int n = s->max_seqlen;
        if (s->cu_seqlens_host) {
            n = s->cu_seqlens_host[b + 1] - s->cu_seqlens_host[b];
            if (n < 1 || n > s->max_seqlen || (b == 0 && s->cu_seqlens_host[0] != 0)) {
                set_error_detail("cu_seqlens: sequence %d has length %d (max_seqlen %d)", b, n, s->max_seqlen);
                return WKV_ERR_SHAPE;
            }
        }
        total += n;
        const int budget = s->budgets_host ? s->budgets_host[b] : s->budget;
        if (budget < 0) {
            set_error_detail("budget of sequence %d is negative (%d)", b, budget);
            return WKV_ERR_BUDGET;
        }
        const int kw = num_windows(n, s->l_obs, s->window);
        const int k = num_selected(n, s->l_obs, s->window, budget);
        if (kw > kw_max) kw_max = kw;
        if (k > k_max) k_max = k;
        if (n - s->l_obs > nr_max) nr_max = n - s->l_obs;
    }
    if (total > 0x7fffffffLL) {
        set_error_detail("more than 2^31-1 tokens in the batch");
        return WKV_ERR_LIMIT;
    }
    ks.batch = s->batch;
    ks.hq = s->n_q_heads;
    ks.hkv = s->n_kv_heads;
    ks.d = s->head_dim;
    ks.alpha = s->l_obs;
    ks.omega = s->window;
    ks.p = s->task == WKV_TASK_LOCALIZATION ? s->window : (s->top_p > 0 ? s->top_p : (s->window + 1) / 2);
    ks.max_seqlen = s->max_seqlen;
    ks.budget = s->budget;
    ks.total_rows = (int)total;
    ks.G = s->n_q_heads / s->n_kv_heads;
    ks.R = ks.G * ks.alpha;
    ks.kw_max = kw_max;
    ks.k_max = k_max;
    ks.nr_max = s->max_seqlen - s->l_obs > 1 ? s->max_seqlen - s->l_obs : 1;
    (void)nr_max;
    {
        const long long cap = (long long)s->l_obs + (long long)kw_max * s->window;
        ks.n_cap = cap < s->max_seqlen ? (int)cap : s->max_seqlen;
    }
    ks.cu = s->cu_seqlens_dev;
    ks.budgets = s->budgets_dev;
    ks.sb = s->stride_b;
    ks.sh = s->stride_h;
    ks.st = s->stride_t;
    ks.qsb = s->q_stride_b;
    ks.qsh = s->q_stride_h;
    ks.qst = s->q_stride_t;
    ks.scale_log2 = (float)(1.4426950408889634 / sqrt((double)s->head_dim));
    return WKV_OK;
}

int check_cuda(cudaError_t e, const char *what)
{
    if (e == cudaSuccess) return WKV_OK;
    set_error_detail("%s: %s", what, cudaGetErrorString(e));
    return WKV_ERR_CUDA;
}

static int check_workspace(const Workspace &ws, const void *workspace, size_t bytes)
{
    if (!workspace) {
        set_error_detail("workspace is NULL (%zu bytes needed)", ws.total);
        return WKV_ERR_WORKSPACE;
    }
    if (bytes < ws.total) {
        set_error_detail("workspace has %zu bytes, %zu needed", bytes, ws.total);
        return WKV_ERR_WORKSPACE;
    }
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) {
        set_error_detail("workspace is not 256-byte aligned");
        return WKV_ERR_WORKSPACE;
    }
    return WKV_OK;
}

// picks the kernel family; returns a status
static int pick_score_impl(const wkv_shape *s, const KShape &ks, const Workspace &ws, bool &use_tc)
{
    const bool tc_ok = score_tc_supported(ks, s->dtype);
    if ((s->score_impl == WKV_SCORE_TCGEN05 || s->score_impl == WKV_SCORE_TCGEN05_PIPELINED) && !tc_ok) {
        set_error_detail("tensor-core score kernels need bf16, head_dim 64/128 and G*alpha <= 256 on a device of "
                         "compute capability 10");
        return WKV_ERR_UNSUPPORTED;
    }
    use_tc = tc_ok && s->score_impl != WKV_SCORE_SIMT;
    if (!use_tc) {
        const size_t need = score_simt_smem_bytes(ks, ws.r_pad);
        if (need > 227u * 1024u) {
            set_error_detail("CUDA-core score kernels need %zu bytes of shared memory (> 227 KB): "
                             "G*alpha*head_dim too large", need);
            return WKV_ERR_UNSUPPORTED;
        }
    }
    return WKV_OK;
}

int do_score(const wkv_shape *s, const KShape &ks, const Workspace &ws, const void *q, const void *k,
             float *window_scores, float *token_scores, int *window_idx, int *kept_len, void *workspace,
             cudaStream_t stream, const float *lse_obs, const PipeGather *gather, bool *gathered)
{
    if (gathered) *gathered = false;
    if (!aligned16(q) || !aligned16(k)) {
        set_error_detail("q_obs / k_leader not 16-byte aligned");
        return WKV_ERR_ALIGN;
    }
    bool use_tc = false;
    int st = pick_score_impl(s, ks, ws, use_tc);
    if (st != WKV_OK) return st;
    if (use_tc) {
        const bool forced = s->score_impl == WKV_SCORE_TCGEN05 || s->score_impl == WKV_SCORE_TCGEN05_PIPELINED;
        st = WKV_ERR_UNSUPPORTED;
        if (s->score_impl == WKV_SCORE_TCGEN05_PIPELINED) {
            if (!group_pipeline_supported(ks, s->dtype)) {
                set_error_detail("the pipelined kernel needs G*alpha <= 128 and observation positions as the faster "
                                 "dimension of Q_obs");
                return WKV_ERR_UNSUPPORTED;
            }
            // one launch for scoring, selection and (when asked and possible) the gather
            const bool fuse = gather && window_idx && group_pipeline_can_gather(ks, elem_bytes(s->dtype), gather->n_tensors);
            st = launch_group_pipeline(ks, q, k, window_scores, token_scores, window_idx, kept_len, workspace, ws,
                                       stream, lse_obs, fuse ? gather : nullptr);
            if (st == WKV_OK && fuse && gathered) *gathered = true;
            return st;
        }
        st = launch_score_tc(ks, q, k, window_scores, token_scores, window_idx, kept_len, workspace, ws, stream,
                                 lse_obs);
        // a key layout that no tensor map can describe is served by the CUDA-core kernels
        if (st != WKV_ERR_UNSUPPORTED || forced) return st;
        if (score_simt_smem_bytes(ks, ws.r_pad) > 227u * 1024u) return st;
    }
    st = check_cuda(launch_score_simt(ks, s->dtype, q, k, window_scores, token_scores, workspace, ws, stream,
                                      lse_obs),
                    "score kernels");
    if (st == WKV_OK && window_idx)
        st = check_cuda(launch_topk(ks, window_scores, window_idx, kept_len, stream), "selection kernel");
    return st;
}

static int fill_table(int n_layers, const void *const *k_layers, const void *const *v_layers,
                      void *const *k_out, void *const *v_out, LayerTable &tab, int &n_tensors)
{
    if (n_layers < 1 || n_layers > WKV_MAX_GROUP_LAYERS) {
        set_error_detail("n_layers %d outside 1..%d", n_layers, WKV_MAX_GROUP_LAYERS);
        return WKV_ERR_LIMIT;
    }
    if (!k_layers || !k_out) {
        set_error_detail("k_layers / k_out_layers is NULL");
        return WKV_ERR_NULL;
    }
    const bool with_v = v_layers && v_out;
    n_tensors = 0;
    for (int l = 0; l < n_layers; ++l) {
        const void *src[2] = {k_layers[l], with_v ? v_layers[l] : nullptr};
        void *dst[2] = {k_out[l], with_v ? v_out[l] : nullptr};
        for (int t = 0; t < (with_v ? 2 : 1); ++t) {
            if (!src[t] || !dst[t]) {
                set_error_detail("layer %d: NULL tensor pointer", l);
                return WKV_ERR_NULL;
            }
            if (!aligned16(src[t]) || !aligned16(dst[t])) {
                set_error_detail("layer %d: tensor pointer not 16-byte aligned", l);
                return WKV_ERR_ALIGN;
            }
            if (src[t] == dst[t]) {
                set_error_detail("layer %d: the compact cache must not be the input tensor itself "
                                 "(wkv_compact_kv_inplace compacts inside one buffer)", l);
                return WKV_ERR_SHAPE;
            }
            tab.src[n_tensors] = src[t];
            tab.dst[n_tensors] = dst[t];
            ++n_tensors;
        }
    }
    return WKV_OK;
}

static int keep_max_of(const wkv_shape *s)
{
    int best = 0;
    for (int b = 0; b < s->batch; ++b) {
        const int n = s->cu_seqlens_host ? s->cu_seqlens_host[b + 1] - s->cu_seqlens_host[b] : s->max_seqlen;
        const int budget = s->budgets_host ? s->budgets_host[b] : s->budget;
        const int rows = num_selected(n, s->l_obs, s->window, budget) * s->window + (n < s->l_obs ? n : s->l_obs);
        if (rows > best) best = rows;
    }
    return best;
}

}  // namespace wkv

using namespace wkv;

extern "C" {

int32_t wkv_num_windows(int32_t n, int32_t alpha, int32_t omega) { return num_windows(n, alpha, omega); }

int32_t wkv_num_selected(int32_t n, int32_t alpha, int32_t omega, int32_t budget)
{
    return num_selected(n, alpha, omega, budget);
}

int32_t wkv_keep_len(int32_t n, int32_t alpha, int32_t omega, int32_t budget, int32_t *k_out)
{
    if (n < 0 || alpha < 1 || omega < 1 || budget < 0) {
        if (k_out) *k_out = 0;
        return -1;
    }
    const int k = num_selected(n, alpha, omega, budget);
    if (k_out) *k_out = k;
    const int n_r = n > alpha ? n - alpha : 0;
    const long long rows = (long long)k * omega;
    // all windows selected: the short last window is among them and the cache is the whole sequence
    return (int32_t)((rows < n_r ? rows : n_r) + (n < alpha ? n : alpha));
}

int wkv_workspace_sync_words(const wkv_shape *s, int32_t unit, size_t *ticket_byte_offset,
                             size_t *arrival_byte_offset)
{
    KShape ks;
    const int st = resolve(s, ks);
    if (st != WKV_OK) return st;
    if (unit < 0 || unit >= ks.batch * ks.hkv) {
        set_error_detail("unit %d outside 0..%d", unit, ks.batch * ks.hkv - 1);
        return WKV_ERR_SHAPE;
    }
    const Workspace ws = plan_workspace(ks);
    const size_t ticket = ws.sync_off + sizeof(int) * ((size_t)kSyncTickets + kSyncWordsPerUnit * (size_t)unit);
    if (ticket_byte_offset) *ticket_byte_offset = ticket;
    if (arrival_byte_offset) *arrival_byte_offset = ticket + sizeof(int);
    return WKV_OK;
}

int32_t wkv_kw_max(const wkv_shape *s)
{
    KShape ks;
    return resolve(s, ks) == WKV_OK ? ks.kw_max : 0;
}

int32_t wkv_k_max(const wkv_shape *s)
{
    KShape ks;
    return resolve(s, ks) == WKV_OK ? ks.k_max : 0;
}

int32_t wkv_keep_max(const wkv_shape *s)
{
    KShape ks;
    return resolve(s, ks) == WKV_OK ? keep_max_of(s) : 0;
}

int wkv_group_budgets(int32_t n_layers, int32_t gamma, int64_t b_total, int32_t lambda_num, int32_t lambda_den,
                      int32_t *per_layer_out)
{
    if (!per_layer_out) {
        set_error_detail("per_layer_out is NULL");
        return WKV_ERR_NULL;
    }
    if (n_layers < 1 || gamma < 1 || n_layers % gamma || b_total < 0 || lambda_den < 1 || lambda_num < lambda_den) {
        set_error_detail("group budgets: n_layers %d, gamma %d, b_total %lld, lambda %d/%d", n_layers, gamma,
                         (long long)b_total, lambda_num, lambda_den);
        return WKV_ERR_SHAPE;
    }
    const int H = n_layers / gamma;
    if (H == 1) {
        per_layer_out[0] = (int32_t)(b_total / gamma);
        return WKV_OK;
    }
    // b^h = T * [(2 num - den)(H - 1) - 2 (num - den) h] / (num * H * (H - 1))   (Eq. 6 into Eq. 7)
    typedef __int128 wide;
    const wide T = b_total, num = lambda_num, den = lambda_den;
    const wide denom = num * H * (H - 1) * gamma;
    wide used = 0;
    for (int h = 0; h < H; ++h) {
        const wide numer = T * ((2 * num - den) * (H - 1) - 2 * (num - den) * h);
        const wide per_layer = numer / denom;     // numer >= 0 because lambda >= 1
        per_layer_out[h] = (int32_t)per_layer;
        used += per_layer * gamma;
    }
    per_layer_out[0] += (int32_t)((T - used) / gamma);
    return WKV_OK;
}

int wkv_jaccard_windows(const int32_t *idx_a, const int32_t *idx_b, int32_t units, int32_t k_max,
                        double *per_unit_out, double *mean_out)
{
    if (!idx_a || !idx_b) {
        set_error_detail("idx_a / idx_b is NULL");
        return WKV_ERR_NULL;
    }
    if (units < 1 || k_max < 1) {
        set_error_detail("jaccard: units %d, k_max %d", units, k_max);
        return WKV_ERR_SHAPE;
    }
    double total = 0.0;
    for (int u = 0; u < units; ++u) {
        const int32_t *a = idx_a + (size_t)u * k_max, *b = idx_b + (size_t)u * k_max;
        int na = 0, nb = 0;
        while (na < k_max && a[na] >= 0) ++na;
        while (nb < k_max && b[nb] >= 0) ++nb;
        for (int i = 1; i < na; ++i)
            if (a[i] <= a[i - 1]) {
                set_error_detail("jaccard: list A of unit %d is not strictly ascending at entry %d", u, i);
                return WKV_ERR_SHAPE;
            }
        for (int i = 1; i < nb; ++i)
            if (b[i] <= b[i - 1]) {
                set_error_detail("jaccard: list B of unit %d is not strictly ascending at entry %d", u, i);
                return WKV_ERR_SHAPE;
            }
        // merge walk over two ascending lists
        int i = 0, j = 0, both = 0;
        while (i < na && j < nb) {
            if (a[i] == b[j]) {
                ++both;
                ++i;
                ++j;
            } else if (a[i] < b[j]) {
                ++i;
            } else {
                ++j;
            }
        }
        const int either = na + nb - both;
        const double jac = either == 0 ? 1.0 : (double)both / (double)either;
        if (per_unit_out) per_unit_out[u] = jac;
        total += jac;
    }
    if (mean_out) *mean_out = total / units;
    return WKV_OK;
}

size_t wkv_workspace_bytes(const wkv_shape *s)
{
    KShape ks;
    if (resolve(s, ks) != WKV_OK) return 0;
    return plan_workspace(ks).total;
}

static int score_windows_entry(const wkv_shape *s, const void *q_obs, const void *k_leader, const float *lse_obs,
                               float *window_scores, float *token_scores, void *workspace,
                               size_t workspace_bytes, void *cuda_stream)
{
    KShape ks;
    int st = resolve(s, ks);
    if (st != WKV_OK) return st;
    if (!q_obs || !k_leader || !window_scores) {
        set_error_detail("q_obs / k_leader / window_scores is NULL");
        return WKV_ERR_NULL;
    }
    const Workspace ws = plan_workspace(ks);
    st = check_workspace(ws, workspace, workspace_bytes);
    if (st != WKV_OK) return st;
    return do_score(s, ks, ws, q_obs, k_leader, window_scores, token_scores, nullptr, nullptr, workspace,
                    static_cast<cudaStream_t>(cuda_stream), lse_obs);
}

int wkv_score_windows(const wkv_shape *s, const void *q_obs, const void *k_leader, float *window_scores,
                      float *token_scores, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    return score_windows_entry(s, q_obs, k_leader, nullptr, window_scores, token_scores, workspace, workspace_bytes,
                               cuda_stream);
}

int wkv_score_windows_lse(const wkv_shape *s, const void *q_obs, const void *k_leader, const float *lse_obs,
                          float *window_scores, float *token_scores, void *workspace, size_t workspace_bytes,
                          void *cuda_stream)
{
    if (!lse_obs) {
        set_error_detail("lse_obs is NULL");
        return WKV_ERR_NULL;
    }
    return score_windows_entry(s, q_obs, k_leader, lse_obs, window_scores, token_scores, workspace, workspace_bytes,
                               cuda_stream);
}

int wkv_select_leader_windows(const wkv_shape *s, const void *q_obs_leader, const void *k_leader,
                              const float *lse_obs, float *window_scores, int32_t *window_idx, int32_t *kept_len,
                              void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    KShape ks;
    int st = resolve(s, ks);
    if (st != WKV_OK) return st;
    if (!q_obs_leader || !k_leader || !window_idx || !kept_len) {
        set_error_detail("q_obs_leader / k_leader / window_idx / kept_len is NULL");
        return WKV_ERR_NULL;
    }
    const Workspace ws = plan_workspace(ks);
    st = check_workspace(ws, workspace, workspace_bytes);
    if (st != WKV_OK) return st;
    float *scores = window_scores ? window_scores
                                  : reinterpret_cast<float *>(static_cast<char *>(workspace) + ws.scores_off);
    return do_score(s, ks, ws, q_obs_leader, k_leader, scores, nullptr, window_idx, kept_len, workspace,
                    static_cast<cudaStream_t>(cuda_stream), lse_obs);
}

int wkv_select_topk_windows(const wkv_shape *s, const float *window_scores, int32_t *window_idx,
                            int32_t *kept_len, void *cuda_stream)
{
    KShape ks;
    int st = resolve(s, ks);
    if (st != WKV_OK) return st;
    if (!window_scores || !window_idx || !kept_len) {
        set_error_detail("window_scores / window_idx / kept_len is NULL");
        return WKV_ERR_NULL;
    }
    return check_cuda(launch_topk(ks, window_scores, window_idx, kept_len, static_cast<cudaStream_t>(cuda_stream)),
                      "selection kernel");
}

int wkv_gather_kv(const wkv_shape *s, int32_t n_layers, const void *const *k_layers,
                  const void *const *v_layers, const int32_t *window_idx, void *const *k_out_layers,
                  void *const *v_out_layers, const int32_t *cu_seqlens_out, int32_t keep_capacity,
                  void *cuda_stream)
{
    KShape ks;
    int st = resolve(s, ks);
    if (st != WKV_OK) return st;
    if (!window_idx) {
        set_error_detail("window_idx is NULL");
        return WKV_ERR_NULL;
    }
    LayerTable tab;
    int n_tensors = 0;
    st = fill_table(n_layers, k_layers, v_layers, k_out_layers, v_out_layers, tab, n_tensors);
    if (st != WKV_OK) return st;
    if (!cu_seqlens_out && keep_capacity < keep_max_of(s)) {
        set_error_detail("keep_capacity %d smaller than the %d rows a unit may keep", keep_capacity, keep_max_of(s));
        return WKV_ERR_SHAPE;
    }
    return check_cuda(launch_gather(ks, elem_bytes(s->dtype), n_tensors, tab, window_idx, cu_seqlens_out,
                                    keep_capacity, static_cast<cudaStream_t>(cuda_stream)),
                      "gather kernel");
}

int wkv_gather_kv_paged(const wkv_shape *s, int32_t n_layers, const void *const *k_layers,
                        const void *const *v_layers, const int32_t *window_idx, void *const *k_pool_layers,
                        void *const *v_pool_layers, const int32_t *block_table, int32_t max_pages,
                        int32_t page_size, int32_t num_pages, int64_t page_stride, int64_t head_stride,
                        int64_t row_stride, void *cuda_stream)
{
    KShape ks;
    int st = resolve(s, ks);
    if (st != WKV_OK) return st;
    if (!window_idx || !block_table) {
        set_error_detail("window_idx / block_table is NULL");
        return WKV_ERR_NULL;
    }
    LayerTable tab;
    int n_tensors = 0;
    st = fill_table(n_layers, k_layers, v_layers, k_pool_layers, v_pool_layers, tab, n_tensors);
    if (st != WKV_OK) return st;
    const int eb = elem_bytes(s->dtype);
    if (max_pages < 1 || page_size < 1 || num_pages < 1 || (long long)max_pages * page_size < keep_max_of(s)) {
        set_error_detail("paged cache: max_pages %d x page_size %d does not cover the %d rows a unit may keep "
                         "(num_pages %d)", max_pages, page_size, keep_max_of(s), num_pages);
        return WKV_ERR_SHAPE;
    }
    const int64_t strides[3] = {page_stride, head_stride, row_stride};
    for (int i = 0; i < 3; ++i)
        if (strides[i] < 0 || (strides[i] * eb) % 16) {
            set_error_detail("paged cache: stride #%d = %lld is negative or not 16-byte aligned", i, (long long)strides[i]);
            return WKV_ERR_ALIGN;
        }
    if (row_stride < s->head_dim) {
        set_error_detail("paged cache: row stride smaller than head_dim");
        return WKV_ERR_SHAPE;
    }
    PagedOut po;
    po.block_table = block_table;
    po.max_pages = max_pages;
    po.page_size = page_size;
    po.num_pages = num_pages;
    po.page_stride = page_stride;
    po.head_stride = head_stride;
    po.row_stride = row_stride;
    return check_cuda(launch_gather(ks, eb, n_tensors, tab, window_idx, nullptr, 0,
                                    static_cast<cudaStream_t>(cuda_stream), &po),
                      "gather kernel (paged output)");
}

int wkv_compact_kv_inplace(const wkv_shape *s, int32_t n_layers, void *const *k_layers, void *const *v_layers,
                           const int32_t *window_idx, void *cuda_stream)
{
    KShape ks;
    int st = resolve(s, ks);
    if (st != WKV_OK) return st;
    if (!window_idx || !k_layers) {
        set_error_detail("window_idx / k_layers is NULL");
        return WKV_ERR_NULL;
    }
    if (n_layers < 1 || n_layers > WKV_MAX_GROUP_LAYERS) {
        set_error_detail("n_layers %d outside 1..%d", n_layers, WKV_MAX_GROUP_LAYERS);
        return WKV_ERR_LIMIT;
    }
    const int eb = elem_bytes(s->dtype);
    if ((long long)s->head_dim * eb > 128 * 1024) {
        set_error_detail("in-place compaction: a row of %lld bytes exceeds 128 KB", (long long)s->head_dim * eb);
        return WKV_ERR_UNSUPPORTED;
    }
    InplaceTable tab;
    int n_tensors = 0;
    for (int l = 0; l < n_layers; ++l) {
        void *p[2] = {k_layers[l], v_layers ? v_layers[l] : nullptr};
        for (int t = 0; t < (v_layers ? 2 : 1); ++t) {
            if (!p[t]) {
                set_error_detail("layer %d: NULL tensor pointer", l);
                return WKV_ERR_NULL;
            }
            if (!aligned16(p[t])) {
                set_error_detail("layer %d: tensor pointer not 16-byte aligned", l);
                return WKV_ERR_ALIGN;
            }
            for (int o = 0; o < n_tensors; ++o)
                if (tab.ptr[o] == p[t]) {
                    set_error_detail("layer %d: the same tensor is listed twice", l);
                    return WKV_ERR_SHAPE;
                }
            tab.ptr[n_tensors++] = p[t];
        }
    }
    return check_cuda(launch_compact_inplace(ks, eb, n_tensors, tab, window_idx, static_cast<cudaStream_t>(cuda_stream)),
                      "in-place compaction kernel");
}

}  // extern "C"

namespace wkv {
uint64_t launches_so_far() { return g_launches.load(std::memory_order_relaxed); }
}  // namespace wkv

int wkv::compress_group_entry(const wkv_shape *s, int32_t n_layers, const void *q_obs_leader, const float *lse_obs,
                                const void *const *k_layers, const void *const *v_layers, void *const *k_out_layers,
                                void *const *v_out_layers, float *window_scores, int32_t *window_idx,
                                int32_t *kept_len, const int32_t *cu_seqlens_out, int32_t keep_capacity,
                                void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    KShape ks;
    int st = resolve(s, ks);
    if (st != WKV_OK) return st;
    if (!q_obs_leader || !window_idx || !kept_len) {
        set_error_detail("q_obs_leader / window_idx / kept_len is NULL");
        return WKV_ERR_NULL;
    }
    LayerTable tab;
    int n_tensors = 0;
    st = fill_table(n_layers, k_layers, v_layers, k_out_layers, v_out_layers, tab, n_tensors);
    if (st != WKV_OK) return st;
    if (!cu_seqlens_out && keep_capacity < keep_max_of(s)) {
        set_error_detail("keep_capacity %d smaller than the %d rows a unit may keep", keep_capacity, keep_max_of(s));
        return WKV_ERR_SHAPE;
    }
    const Workspace ws = plan_workspace(ks);
    st = check_workspace(ws, workspace, workspace_bytes);
    if (st != WKV_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    float *scores = window_scores ? window_scores
                                  : reinterpret_cast<float *>(static_cast<char *>(workspace) + ws.scores_off);
    PipeGather pg;
    pg.n_tensors = n_tensors;
    pg.tab = &tab;
    pg.cu_out = cu_seqlens_out;
    pg.keep_capacity = keep_capacity;
    bool gathered = false;
    st = do_score(s, ks, ws, q_obs_leader, k_layers[0], scores, nullptr, window_idx, kept_len, workspace, stream,
                  lse_obs, &pg, &gathered);
    if (st != WKV_OK || gathered) return st;
    return check_cuda(launch_gather(ks, elem_bytes(s->dtype), n_tensors, tab, window_idx, cu_seqlens_out,
                                    keep_capacity, stream),
                      "gather kernel");
}

extern "C" {

int wkv_compress_group(const wkv_shape *s, int32_t n_layers, const void *q_obs_leader,
                       const void *const *k_layers, const void *const *v_layers, void *const *k_out_layers,
                       void *const *v_out_layers, float *window_scores, int32_t *window_idx,
                       int32_t *kept_len, const int32_t *cu_seqlens_out, int32_t keep_capacity,
                       void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    return compress_group_entry(s, n_layers, q_obs_leader, nullptr, k_layers, v_layers, k_out_layers, v_out_layers,
                                window_scores, window_idx, kept_len, cu_seqlens_out, keep_capacity, workspace,
                                workspace_bytes, cuda_stream);
}

int wkv_compress_group_lse(const wkv_shape *s, int32_t n_layers, const void *q_obs_leader, const float *lse_obs,
                           const void *const *k_layers, const void *const *v_layers, void *const *k_out_layers,
                           void *const *v_out_layers, float *window_scores, int32_t *window_idx,
                           int32_t *kept_len, const int32_t *cu_seqlens_out, int32_t keep_capacity,
                           void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!lse_obs) {
        set_error_detail("lse_obs is NULL");
        return WKV_ERR_NULL;
    }
    return compress_group_entry(s, n_layers, q_obs_leader, lse_obs, k_layers, v_layers, k_out_layers, v_out_layers,
                                window_scores, window_idx, kept_len, cu_seqlens_out, keep_capacity, workspace,
                                workspace_bytes, cuda_stream);
}

int wkv_compress_group_host(const wkv_shape *s, int32_t n_layers, const void *q_obs_host, size_t q_bytes,
                            const void *const *k_layers_host, const void *const *v_layers_host,
                            size_t bytes_per_layer, void *const *k_out_layers_host,
                            void *const *v_out_layers_host, size_t out_bytes_per_layer,
                            int32_t *window_idx_host, int32_t *kept_len_host, void *q_obs_dev,
                            void *const *k_layers_dev, void *const *v_layers_dev,
                            void *const *k_out_layers_dev, void *const *v_out_layers_dev,
                            int32_t *window_idx_dev, int32_t *kept_len_dev, int32_t keep_capacity,
                            void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    KShape ks;
    int st = resolve(s, ks);
    if (st != WKV_OK) return st;
    if (n_layers < 1 || n_layers > WKV_MAX_GROUP_LAYERS) {
        set_error_detail("n_layers %d outside 1..%d", n_layers, WKV_MAX_GROUP_LAYERS);
        return WKV_ERR_LIMIT;
    }
    if (!q_obs_host || !k_layers_host || !v_layers_host || !k_out_layers_host || !v_out_layers_host ||
        !window_idx_host || !kept_len_host || !q_obs_dev || !k_layers_dev || !v_layers_dev ||
        !k_out_layers_dev || !v_out_layers_dev || !window_idx_dev || !kept_len_dev) {
        set_error_detail("a host or staging pointer is NULL");
        return WKV_ERR_NULL;
    }
    // the byte counts are the caller's: they must cover what the shape says the kernels will touch,
    // and the output count must be exactly one dense compact cache
    {
        const size_t eb = (size_t)elem_bytes(s->dtype);
        const size_t rows = ks.cu ? (size_t)ks.total_rows : (size_t)ks.max_seqlen;
        const size_t kv_extent = ((rows - 1) * (size_t)ks.st + (size_t)(ks.batch - 1) * (size_t)ks.sb +
                                  (size_t)(ks.hkv - 1) * (size_t)ks.sh + (size_t)ks.d) * eb;
        const size_t q_extent = ((size_t)(ks.batch - 1) * (size_t)ks.qsb + (size_t)(ks.hq - 1) * (size_t)ks.qsh +
                                 (size_t)(ks.alpha - 1) * (size_t)ks.qst + (size_t)ks.d) * eb;
        if (bytes_per_layer < kv_extent || q_bytes < q_extent) {
            set_error_detail("host buffers smaller than the shape: bytes_per_layer %zu (needs %zu), q_bytes %zu "
                             "(needs %zu)", bytes_per_layer, kv_extent, q_bytes, q_extent);
            return WKV_ERR_SHAPE;
        }
        if (keep_capacity < keep_max_of(s)) {
            set_error_detail("keep_capacity %d smaller than the %d rows a unit may keep", keep_capacity,
                             keep_max_of(s));
            return WKV_ERR_SHAPE;
        }
        const size_t out_exact = (size_t)ks.batch * ks.hkv * (size_t)keep_capacity * ks.d * eb;
        if (out_bytes_per_layer != out_exact) {
            set_error_detail("out_bytes_per_layer %zu is not one dense compact cache [B, H_kv, keep_capacity, d] "
                             "= %zu bytes", out_bytes_per_layer, out_exact);
            return WKV_ERR_SHAPE;
        }
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // The copies in dominate this call, so it is laid out as a pipeline over the layers: the leader's
    // keys go first and are scored as soon as they have landed; every layer is gathered behind its own
    // copy in, and its compact cache travels back on a second stream while the next layer is still
    // coming in (the two copy directions run at the same time).
    cudaStream_t back = nullptr;
    cudaEvent_t ready = nullptr;
    st = check_cuda(cudaStreamCreateWithFlags(&back, cudaStreamNonBlocking), "stream for the copies back");
    if (st != WKV_OK) return st;
    st = check_cuda(cudaEventCreateWithFlags(&ready, cudaEventDisableTiming), "event");
    const size_t units = (size_t)ks.batch * ks.hkv;
    auto h2d = [&](void *dst, const void *src, size_t bytes, const char *what) {
        if (st == WKV_OK) st = check_cuda(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, stream), what);
    };
    auto d2h_after = [&](void *dst, const void *src, size_t bytes, const char *what) {
        if (st == WKV_OK) st = check_cuda(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, back), what);
    };
    auto hand_over = [&]() {     // what `stream` has done so far precedes what `back` does next
        if (st == WKV_OK) st = check_cuda(cudaEventRecord(ready, stream), "event record");
        if (st == WKV_OK) st = check_cuda(cudaStreamWaitEvent(back, ready, 0), "event wait");
    };
    h2d(q_obs_dev, q_obs_host, q_bytes, "copy of q_obs");
    h2d(k_layers_dev[0], k_layers_host[0], bytes_per_layer, "copy of K");
    if (st == WKV_OK)
        st = wkv_select_leader_windows(s, q_obs_dev, k_layers_dev[0], nullptr, nullptr, window_idx_dev, kept_len_dev,
                                       workspace, workspace_bytes, cuda_stream);
    hand_over();
    d2h_after(window_idx_host, window_idx_dev, units * ks.k_max * sizeof(int32_t), "copy of window_idx");
    d2h_after(kept_len_host, kept_len_dev, units * sizeof(int32_t), "copy of kept_len");
    for (int l = 0; l < n_layers && st == WKV_OK; ++l) {
        if (l > 0) h2d(k_layers_dev[l], k_layers_host[l], bytes_per_layer, "copy of K");
        h2d(v_layers_dev[l], v_layers_host[l], bytes_per_layer, "copy of V");
        if (st == WKV_OK)
            st = wkv_gather_kv(s, 1, k_layers_dev + l, v_layers_dev + l, window_idx_dev, k_out_layers_dev + l,
                               v_out_layers_dev + l, nullptr, keep_capacity, cuda_stream);
        hand_over();
        d2h_after(k_out_layers_host[l], k_out_layers_dev[l], out_bytes_per_layer, "copy of compact K");
        d2h_after(v_out_layers_host[l], v_out_layers_dev[l], out_bytes_per_layer, "copy of compact V");
    }
    // both streams are drained before the call returns, whatever happened above
    const cudaError_t e1 = cudaStreamSynchronize(stream), e2 = cudaStreamSynchronize(back);
    if (ready) cudaEventDestroy(ready);
    cudaStreamDestroy(back);
    if (st != WKV_OK) return st;
    if (e1 != cudaSuccess) return check_cuda(e1, "stream synchronisation");
    return check_cuda(e2, "stream synchronisation (copies back)");
}

const char *wkv_status_string(int status)
{
    switch (status) {
    case WKV_OK: return "ok";
    case WKV_ERR_NULL: return "required pointer is NULL";
    case WKV_ERR_SHAPE: return "invalid shape";
    case WKV_ERR_DTYPE: return "invalid dtype";
    case WKV_ERR_BUDGET: return "invalid budget";
    case WKV_ERR_WORKSPACE: return "workspace missing, too small or misaligned";
    case WKV_ERR_ALIGN: return "pointer or stride not 16-byte aligned";
    case WKV_ERR_UNSUPPORTED: return "shape not supported by the kernels";
    case WKV_ERR_CUDA: return "CUDA call failed";
    case WKV_ERR_LIMIT: return "size beyond a fixed maximum";
    default: return "unknown status";
    }
}

const char *wkv_last_error_detail(void) { return g_detail; }

uint64_t wkv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
