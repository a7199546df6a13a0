/*
 * wkv — WindowKV prefill-time KV-cache window selection for NVIDIA B200 (sm_100a).
 *
 * C ABI of the library.  Notation follows the paper (section 2.2.1 / 2.2.2):
 *   n      context length of a sequence (observation window included)
 *   alpha  observation-window length   (field l_obs)
 *   omega  review-window length        (field window)
 *   p      Top-p count of Eq. 4        (field top_p, aggregation task only)
 *   gamma  layers per group            (argument n_layers)
 *   b      per-layer KV budget in tokens, observation window included
 *   G      query heads per KV head = n_q_heads / n_kv_heads
 * A "unit" is one (sequence, KV head) pair.  Derived integers, identical on
 * host and device:
 *   K_w = ceil((n - alpha)/omega)  (0 when n <= alpha)          — Eq. 3
 *   k   = min(K_w, max(0, floor((b - alpha)/omega)))            — budget sentence after Eq. 4
 *
 * General conventions
 *   - Every pointer marked DEVICE is device memory owned by the caller; HOST
 *     pointers are ordinary host memory read before the function returns.
 *     The library allocates and frees nothing and keeps no state between
 *     calls other than a launch counter.
 *   - All device work is enqueued on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and the functions return
 *     without synchronising.
 *   - Argument errors are detected on the host before anything is enqueued
 *     and returned as a wkv_status (0 = success).  wkv_last_error_detail()
 *     gives a thread-local human-readable reason for the last failure.
 *   - Tensors have the head dimension contiguous.  K/V element (b, h, j, c)
 *     lives at  base[(off_b + j)*stride_t + b*stride_b + h*stride_h + c]
 *     where off_b = cu_seqlens[b] for the packed layout (then stride_b = 0)
 *     and 0 for the dense layout.  Dense [B,H_kv,N,d]:
 *     stride_b = H_kv*N*d, stride_h = N*d, stride_t = d.  Packed [T,H_kv,d]:
 *     stride_b = 0, stride_h = d, stride_t = H_kv*d.
 *     Q_obs element (b, hq, i, c) at q[b*q_stride_b + hq*q_stride_h + i*q_stride_t + c],
 *     i = 0..alpha-1 being positions n-alpha .. n-1 of the sequence.
 *   - Base pointers and row strides must be 16-byte aligned.
 *   - cu_seqlens and budgets exist twice, as a HOST and as a DEVICE array.  Sizes of outputs and
 *     of the workspace are derived from the host copies, the kernels read the device copies: the
 *     two must hold the same values when a call is made.  The library does not compare them.  As a
 *     guard, the kernels take no sequence to be longer and no selection to be larger than the host
 *     copies allowed for, so a stale device copy gives wrong results, not accesses outside the
 *     arrays sized from the host copy.
 *   - No output may overlap an input of the same call: the gather reads K/V through the
 *     read-only data path while other warps are already writing the compact cache, so compacting
 *     a tensor into its own front (k_out[l] == k_layers[l]) gives undefined rows.
 *     wkv_gather_kv and the group calls refuse identical input and output pointers of a layer
 *     (WKV_ERR_SHAPE); partial overlaps are the caller's to avoid.  wkv_compact_kv_inplace is the
 *     entry point for compaction inside one buffer.
 */
#ifndef WKV_H_
#define WKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    WKV_OK = 0,
    WKV_ERR_NULL = 1,        /* a required pointer is NULL */
    WKV_ERR_SHAPE = 2,       /* inconsistent or non-positive sizes */
    WKV_ERR_DTYPE = 3,
    WKV_ERR_BUDGET = 4,      /* negative budget */
    WKV_ERR_WORKSPACE = 5,   /* workspace missing, too small or misaligned */
    WKV_ERR_ALIGN = 6,       /* pointer or stride not 16-byte aligned */
    WKV_ERR_UNSUPPORTED = 7, /* shape outside what the kernels cover */
    WKV_ERR_CUDA = 8,        /* a CUDA runtime / driver call failed */
    WKV_ERR_LIMIT = 9        /* size beyond a documented fixed maximum */
} wkv_status;

typedef enum { WKV_F32 = 0, WKV_BF16 = 1 } wkv_dtype;
typedef enum { WKV_TASK_LOCALIZATION = 0, WKV_TASK_AGGREGATION = 1 } wkv_task;
/* which score kernel family to use: AUTO picks the tensor-core (tcgen05) kernels
 * for bf16 inputs with head_dim 64 or 128 and G*alpha <= 256, else the plain
 * CUDA-core kernels.  TCGEN05 forces the tensor-core kernels (score + selection in one launch,
 * the gather in a second one).  TCGEN05_PIPELINED asks for the single-launch form instead
 * (G*alpha <= 128 only): statistics sweep one wave ahead of the scoring sweep and the gather done
 * by bulk copies inside the same kernel.  It gives the same results and is slower on every
 * configuration measured so far, so AUTO never picks it; it is kept as an option for
 * measurements. */
typedef enum { WKV_SCORE_AUTO = 0, WKV_SCORE_SIMT = 1, WKV_SCORE_TCGEN05 = 2, WKV_SCORE_TCGEN05_PIPELINED = 3 } wkv_score_impl;

#define WKV_MAX_GROUP_LAYERS 32

typedef struct {
    uint32_t struct_size;   /* sizeof(wkv_shape), checked */
    int32_t dtype;          /* wkv_dtype of Q, K, V and of the compact cache */
    int32_t batch;          /* B */
    int32_t n_q_heads;      /* H_q, a multiple of n_kv_heads */
    int32_t n_kv_heads;     /* H_kv */
    int32_t head_dim;       /* d, a multiple of 8 (bf16) / 4 (fp32) */
    int32_t l_obs;          /* alpha >= 1 */
    int32_t window;         /* omega >= 1 */
    int32_t top_p;          /* p for WKV_TASK_AGGREGATION; 0 => ceil(omega/2) */
    int32_t task;           /* wkv_task: selects p = omega (localization) or p = top_p */
    int32_t max_seqlen;     /* N: the common length (dense) or an upper bound (packed) */
    int32_t budget;         /* per-layer budget b for every sequence, used when budgets_host == NULL */
    int32_t score_impl;     /* wkv_score_impl */
    int32_t reserved;       /* must be 0 */
    const int32_t *cu_seqlens_host; /* HOST  [B+1] or NULL => dense, every n_b = max_seqlen */
    const int32_t *cu_seqlens_dev;  /* DEVICE copy of the same array (required iff the host one is given) */
    const int32_t *budgets_host;    /* HOST  [B] per-sequence budgets, or NULL => `budget` */
    const int32_t *budgets_dev;     /* DEVICE copy of the same array (required iff the host one is given) */
    int64_t stride_b, stride_h, stride_t;       /* K/V element strides */
    int64_t q_stride_b, q_stride_h, q_stride_t; /* Q_obs element strides */
} wkv_shape;

/* ---- host-side integer helpers (Eq. 3 and the budget sentence after Eq. 4) ---- */
int32_t wkv_num_windows(int32_t n, int32_t alpha, int32_t omega);                   /* K_w */
int32_t wkv_num_selected(int32_t n, int32_t alpha, int32_t omega, int32_t budget);  /* k   */
/* Rows of one unit's compact cache and, through *k_out (may be NULL), the number k of selected
 * windows, for a sequence of n tokens: min(k*omega, n - alpha) + min(alpha, n).  This is the
 * capacity to provide; a unit keeps (omega - size of the last window) rows fewer when k < K_w and
 * the short last window of the sequence is among the selected ones (kept_len reports the exact
 * count).  Returns -1 for negative n / budget or alpha, omega < 1. */
int32_t wkv_keep_len(int32_t n, int32_t alpha, int32_t omega, int32_t budget, int32_t *k_out);
/* Leading sizes of the output arrays for a whole batch: */
int32_t wkv_kw_max(const wkv_shape *s);   /* max_b K_w,b, at least 1 */
int32_t wkv_k_max(const wkv_shape *s);    /* max_b k_b,   at least 1 */
int32_t wkv_keep_max(const wkv_shape *s); /* max_b (k_b*omega + min(alpha, n_b)): row capacity of the dense compact cache */

/*
 * Dynamic (pyramid) budget allocation, Eq. 5-7: the H = n_layers / gamma groups get budgets in an
 * arithmetic sequence from b^0 (bottom group) down to b^{H-1} = b_total / (lambda * H) (top group),
 * b^0 = 2 * b_total / H - b^{H-1}, and each group's budget is split evenly over its gamma layers.
 * lambda = lambda_num / lambda_den (the paper uses 14) is taken as a ratio of integers so that the
 * result is exact: out[h] = floor(b^h / gamma) tokens per layer of group h, and the tokens lost to
 * the flooring go, in whole multiples of gamma, to group 0.  The per-layer values are what the
 * `budget` / `budgets_host` fields of wkv_shape expect.  Host function, no device work.
 *   b_total         total budget over all layers (e.g. n_layers * average per-layer budget)
 *   per_layer_out   HOST out, int32 [n_layers / gamma]
 * Returns WKV_ERR_SHAPE for n_layers % gamma != 0, lambda < 1 or non-positive sizes.
 */
int wkv_group_budgets(int32_t n_layers, int32_t gamma, int64_t b_total, int32_t lambda_num, int32_t lambda_den,
                      int32_t *per_layer_out);

/*
 * Jaccard similarity of retained-window index sets (section 3.2, the intra-group similarity the
 * index sharing of section 2.2.2 rests on): |A n B| / |A u B| per unit for two selections of the same
 * batch, e.g. the lists two different layers would select.  Host function on HOST arrays, no device
 * work.
 *   idx_a, idx_b   HOST int32 [units, k_max]: ascending window indices, padded with negative entries
 *                  (the layout wkv_select_topk_windows writes, copied to the host)
 *   per_unit_out   HOST out or NULL, double [units]; two empty sets count as identical (1.0)
 *   mean_out       HOST out or NULL: the mean over the units
 * Returns WKV_ERR_SHAPE for non-positive sizes or a list that is not strictly ascending.
 */
int wkv_jaccard_windows(const int32_t *idx_a, const int32_t *idx_b, int32_t units, int32_t k_max,
                        double *per_unit_out, double *mean_out);

/* Bytes of DEVICE scratch that wkv_score_windows / wkv_compress_group need for this
 * shape (256-byte aligned base expected).  Returns 0 for an invalid shape. */
size_t wkv_workspace_bytes(const wkv_shape *s);

/* Byte offsets, inside the workspace of this shape, of the two words through which the blocks of a
 * launch synchronise on `unit` (a ticket count and a count of arrived statistics chunks; both are
 * zero between launches).  Diagnostic helper (no counterpart in the paper): lets a test or a
 * debugger inspect or disturb the hand-over without knowing the workspace layout.  Either output
 * may be NULL.  The status word is always at byte 0. */
int wkv_workspace_sync_words(const wkv_shape *s, int32_t unit, size_t *ticket_byte_offset,
                             size_t *arrival_byte_offset);

/*
 * Eq. 1-4 for the group's leader layer.
 * For every unit: logits of the G*alpha observation rows against every key the row
 * may attend to (causal: keys 0..position), softmax per row (Eq. 1), sum over the
 * rows and the G heads for each review token j < n - alpha (Eq. 2), then the
 * window score s_k = sum(Top-p of window k)/min(p, |window k|) (Eq. 3-4; the last
 * window may be shorter than omega).  fp32 accumulation throughout.
 *   q_obs          DEVICE  observation queries of the leader
 *   k_leader       DEVICE  keys of the leader
 *   window_scores  DEVICE  out, float [B, H_kv, wkv_kw_max()] ; entries >= K_w,b are not written
 *   token_scores   DEVICE  out or NULL, float [B, H_kv, max(1, max_seqlen - alpha)] ; t_j of Eq. 2
 *   workspace      DEVICE  scratch of wkv_workspace_bytes() bytes.  Zero it once after allocating
 *                  it.  Its first int32 is a status word that the kernels only ever OR into
 *                  (bit 0: a bounded wait inside a kernel expired, results invalid); the words
 *                  behind it synchronise the blocks of a launch and reset themselves when the
 *                  launch ends normally.  After a non-zero status zero the workspace again.
 *                  One workspace serves one launch at a time.
 */
int wkv_score_windows(const wkv_shape *s, const void *q_obs, const void *k_leader,
                      float *window_scores, float *token_scores,
                      void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * The same stage for callers that cannot allocate device memory (no counterpart in the paper: an
 * engineering variant).  A serving engine that gave all of HBM to its own cache pool at start-up,
 * or code running where cudaMalloc is forbidden, has no way to provide the workspace above; here
 * the scratch is a fixed area of WKV_STATIC_SCRATCH_BYTES inside the library image, which every
 * GPU that loads the library holds until the process exits.  The function allocates and frees
 * nothing.
 *   - Shapes whose wkv_workspace_bytes() exceeds WKV_STATIC_SCRATCH_BYTES are refused with
 *     WKV_ERR_LIMIT before anything is enqueued.
 *   - The first call on each device looks up the area's device address (with that device current);
 *     make that first call outside any stream capture.
 *   - All calls on a device share the one area: two calls whose kernels may overlap on the GPU
 *     (different streams, no dependency) race on it.  Every call first clears the status and
 *     synchronisation words at the head of the area, so an overlapping call does more than
 *     corrupt scores: it wipes the arrival counts of the kernel already running, whose blocks
 *     then sit in their bounded waits for one to two seconds and end with status bit 0 set (in
 *     either call); the scores of both calls are invalid.  Calls on one stream are safe.
 *   - The looked-up address belongs to the device's primary context; after cudaDeviceReset() in
 *     this process the entry point must not be used again.
 *   - device_status  DEVICE out or NULL: receives 0, or the error bits a kernel set
 *     (1 = a bounded wait inside a kernel expired and the scores are invalid).
 * Other arguments and results exactly as wkv_score_windows.
 */
#define WKV_STATIC_SCRATCH_BYTES (4u << 20)
int wkv_score_windows_static(const wkv_shape *s, const void *q_obs, const void *k_leader,
                             float *window_scores, float *token_scores, int32_t *device_status,
                             void *cuda_stream);

/*
 * Budgeted selection (sentence after Eq. 4): per unit the k highest window scores,
 * ties to the lower window index, indices written in ascending order.
 *   window_scores  DEVICE  in,  float [B, H_kv, wkv_kw_max()]
 *   window_idx     DEVICE  out, int32 [B, H_kv, wkv_k_max()], entries >= k_b set to -1
 *   kept_len       DEVICE  out, int32 [B, H_kv]: rows of the compact cache of the unit
 *                  (tokens in the selected windows + min(alpha, n_b))
 */
int wkv_select_topk_windows(const wkv_shape *s, const float *window_scores,
                            int32_t *window_idx, int32_t *kept_len, void *cuda_stream);

/*
 * Intra-group index sharing (section 2.2.2): builds the compact cache of n_layers
 * layers from one set of window indices.  Output row r of a unit is source row
 * idx[r/omega]*omega + r%omega for the retained review rows (ascending position),
 * followed by the observation rows n-alpha .. n-1.  Bit copies.
 *   k_layers, v_layers          HOST arrays [n_layers] of DEVICE pointers (inputs, layout of `s`)
 *   k_out_layers, v_out_layers  HOST arrays [n_layers] of DEVICE pointers (outputs)
 *   window_idx                  DEVICE int32 [B, H_kv, wkv_k_max()] as written by the selection; an entry
 *                               outside [0, K_w) among a unit's first k is skipped (its rows of the
 *                               output are left as they are), never followed
 *   cu_seqlens_out              DEVICE int32 [B+1] or NULL.
 *       NULL  => dense output [B, H_kv, keep_capacity, d]; rows >= kept_len are not written.
 *       else  => packed output [T_out, H_kv, d], sequence b starting at row cu_seqlens_out[b].
 *   keep_capacity               rows per unit of the dense output (>= wkv_keep_max()); ignored when packed
 * Either of v_layers / v_out_layers may be NULL to gather keys only.
 */
int wkv_gather_kv(const wkv_shape *s, int32_t n_layers,
                  const void *const *k_layers, const void *const *v_layers,
                  const int32_t *window_idx,
                  void *const *k_out_layers, void *const *v_out_layers,
                  const int32_t *cu_seqlens_out, int32_t keep_capacity, void *cuda_stream);

/*
 * The same gather into a PAGED compact cache (section 2.2.2; the cache that the decode phase of
 * section 2.1 attends over, in the block-table form serving engines keep it in).  Row r of unit (b, h)
 * goes to page block_table[b][r / page_size], slot r % page_size; pool element (page, h, slot, c) lives
 * at  pool[page*page_stride + h*head_stride + slot*row_stride + c]  (e.g. [pages, H_kv, page_size, d]:
 * page_stride = H_kv*page_size*d, head_stride = page_size*d, row_stride = d; token-major pages
 * [pages, page_size, H_kv, d]: head_stride = d, row_stride = H_kv*d).  One block table serves every
 * layer and both K and V, as the index sharing of the group implies; per-unit lengths are kept_len.
 *   k_pool_layers, v_pool_layers   HOST arrays [n_layers] of DEVICE pool pointers (v may be NULL with v_layers)
 *   block_table   DEVICE int32 [B, max_pages]; an entry outside [0, num_pages) makes its rows be skipped
 *   max_pages * page_size must cover wkv_keep_max(); strides in elements, multiples of 16 bytes
 * Other arguments as wkv_gather_kv.
 */
int wkv_gather_kv_paged(const wkv_shape *s, int32_t n_layers,
                        const void *const *k_layers, const void *const *v_layers,
                        const int32_t *window_idx,
                        void *const *k_pool_layers, void *const *v_pool_layers,
                        const int32_t *block_table, int32_t max_pages, int32_t page_size, int32_t num_pages,
                        int64_t page_stride, int64_t head_stride, int64_t row_stride, void *cuda_stream);

/*
 * Compaction in place (section 2.2.2 as it is driven during prefill: a layer's compact cache takes the
 * place of its full K/V).  For every layer tensor and every unit, the retained rows (selected windows
 * in ascending position, then the observation rows) are moved to the front of the unit's own rows,
 * in the tensor's own layout: afterwards row r < kept_len of unit (b, h) holds what wkv_gather_kv would
 * have written to row r of the compact cache; rows from kept_len on hold leftovers.  Rows only move
 * toward lower addresses; the kernel orders the reads of a stretch of rows before the writes that land
 * on them (one thread block walks a unit's rows in ascending batches), so the result is exact.
 *   k_layers, v_layers   HOST arrays [n_layers] of DEVICE pointers, read AND written (v_layers may be NULL)
 *   window_idx           DEVICE int32 [B, H_kv, wkv_k_max()], an ascending selection as written by
 *                        wkv_select_topk_windows; entries that are no window of the sequence or lie
 *                        before their own slot are skipped (their rows stay as they are)
 * A row of head_dim elements may be at most 128 KB.
 */
int wkv_compact_kv_inplace(const wkv_shape *s, int32_t n_layers, void *const *k_layers, void *const *v_layers,
                           const int32_t *window_idx, void *cuda_stream);

/*
 * One layer group (sections 2.2.1-2.2.2): score + select on k_layers[0] with q_obs_leader,
 * then the shared-index gather of all n_layers layers.  Arguments as above;
 * window_scores may be NULL (then the scores live in the workspace only).
 */
int wkv_compress_group(const wkv_shape *s, int32_t n_layers, const void *q_obs_leader,
                       const void *const *k_layers, const void *const *v_layers,
                       void *const *k_out_layers, void *const *v_out_layers,
                       float *window_scores, int32_t *window_idx, int32_t *kept_len,
                       const int32_t *cu_seqlens_out, int32_t keep_capacity,
                       void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Scoring and the whole group for callers that already hold Eq. 1's normalisers.  The prefill
 * attention of the leader layer computes, for every query row, the log-sum-exp of its causal
 * softmax; handing in the values of the observation rows removes the pass over the keys that
 * otherwise recomputes them (the keys are then read once and never re-read).
 *   lse_obs   DEVICE float [B, H_q, alpha], contiguous: natural log of
 *             sum_{j <= position(i)} exp(q_i . k_j / sqrt(d)) for observation row i of query
 *             head h (row i of head h at (b * H_q + h) * alpha + i), over ALL keys the row may
 *             attend to, observation-window keys included (Eq. 1's denominator).
 * Everything else as in wkv_score_windows / wkv_compress_group.  Values that are not the
 * normalisers of q_obs and k_leader give scores that are wrong by the corresponding factor per
 * row; nothing checks them.  NULL lse_obs is an error (WKV_ERR_NULL).
 */
int wkv_score_windows_lse(const wkv_shape *s, const void *q_obs, const void *k_leader,
                          const float *lse_obs, float *window_scores, float *token_scores,
                          void *workspace, size_t workspace_bytes, void *cuda_stream);
int wkv_compress_group_lse(const wkv_shape *s, int32_t n_layers, const void *q_obs_leader,
                           const float *lse_obs,
                           const void *const *k_layers, const void *const *v_layers,
                           void *const *k_out_layers, void *const *v_out_layers,
                           float *window_scores, int32_t *window_idx, int32_t *kept_len,
                           const int32_t *cu_seqlens_out, int32_t keep_capacity,
                           void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Layer-by-layer use (section 2.2.2: the leader's indices serve the whole group).  During prefill
 * the layers of a group appear one after the other: call this on the leader layer as soon as its
 * keys exist (scores, pooling and selection in one launch on the tensor-core path, nothing
 * gathered), keep window_idx, and call wkv_gather_kv with n_layers = 1 on the leader and on every
 * follower layer when its K/V have been written.  The result equals wkv_compress_group on the
 * same tensors.
 *   lse_obs        DEVICE float [B, H_q, alpha] as in wkv_score_windows_lse, or NULL (then the
 *                  normalisers are computed here)
 *   window_scores  DEVICE out or NULL (then the scores live in the workspace only)
 *   window_idx, kept_len, workspace   as in wkv_compress_group
 */
int wkv_select_leader_windows(const wkv_shape *s, const void *q_obs_leader, const void *k_leader,
                              const float *lse_obs, float *window_scores,
                              int32_t *window_idx, int32_t *kept_len,
                              void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * A layer group as a replayable object (sections 2.2.1-2.2.2, the same computation as
 * wkv_compress_group / wkv_compress_group_lse).  For engines that call the group with the same
 * buffers again and again (static K/V pools and compact caches): create records the launches of
 * the call in a CUDA graph once, launch replays it on a stream, which leaves a smaller gap at the
 * kernel boundary than separate launches do.  The plan owns only the graph; every buffer stays
 * the caller's and must stay valid and at its address for as long as the plan is launched.  What a
 * launch computes depends on the buffers' contents at that moment only.
 *   create   arguments as wkv_compress_group_lse (lse_obs may be NULL: then the normalisers are
 *            computed); validates as the direct call does and launches nothing.  Host-side
 *            resources (a graph) are allocated; no device buffer of the caller's is touched.
 *            `budgets` and the strides of `s` are read now, not at launch.
 *   launch   enqueues the group on cuda_stream; one plan is in flight once at a time (it uses
 *            the one workspace it was created with).
 *   destroy  after the last launch has completed.  NULL is ignored.
 */
typedef struct wkv_group_plan wkv_group_plan;
int wkv_group_plan_create(const wkv_shape *s, int32_t n_layers, const void *q_obs_leader,
                          const float *lse_obs,
                          const void *const *k_layers, const void *const *v_layers,
                          void *const *k_out_layers, void *const *v_out_layers,
                          float *window_scores, int32_t *window_idx, int32_t *kept_len,
                          const int32_t *cu_seqlens_out, int32_t keep_capacity,
                          void *workspace, size_t workspace_bytes, wkv_group_plan **plan_out);
int wkv_group_plan_launch(wkv_group_plan *plan, void *cuda_stream);
void wkv_group_plan_destroy(wkv_group_plan *plan);

/*
 * The same group with every tensor in HOST memory (pinned memory recommended): the
 * inputs are copied to caller-provided DEVICE staging buffers, the group is
 * compressed there, and indices, kept lengths and the compact caches are copied
 * back; the function returns after everything it enqueued has completed.  The copies
 * dominate, so the call runs as a pipeline over the layers: the leader's keys first
 * (scored and selected as soon as they have landed), then layer by layer copy in, gather,
 * and copy back on a second stream of the call's own, so that both copy directions are
 * busy at once.  (This creates and destroys one stream and one event per call.)
 *   *_host arguments    HOST pointers / HOST arrays of HOST pointers
 *   *_dev arguments     DEVICE staging of the same sizes (HOST arrays of DEVICE pointers)
 *   bytes_per_layer     size of one K (or V) tensor; out_bytes_per_layer of one compact cache
 * Dense output layout only.
 */
int wkv_compress_group_host(const wkv_shape *s, int32_t n_layers,
                            const void *q_obs_host, size_t q_bytes,
                            const void *const *k_layers_host, const void *const *v_layers_host,
                            size_t bytes_per_layer,
                            void *const *k_out_layers_host, void *const *v_out_layers_host,
                            size_t out_bytes_per_layer,
                            int32_t *window_idx_host, int32_t *kept_len_host,
                            void *q_obs_dev, void *const *k_layers_dev, void *const *v_layers_dev,
                            void *const *k_out_layers_dev, void *const *v_out_layers_dev,
                            int32_t *window_idx_dev, int32_t *kept_len_dev, int32_t keep_capacity,
                            void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Measurement aid (no counterpart in the paper): launches a kernel that does nothing but evaluate
 * ex2.approx.ftz.f32 (the exponential of Eq. 1 in base 2, the instruction that bounds the score
 * stage) in eight independent chains per thread, `iters` times.  Timing the launch with CUDA events
 * and dividing *ex2_per_launch by it gives the device's rate for that instruction, which the
 * benchmark uses as the special-function floor of the score kernels.
 *   scratch_dev     DEVICE float[1] (never written in practice)
 *   blocks, threads grid and block size (threads a multiple of 32, at most 1024)
 *   ex2_per_launch  HOST out or NULL: exponentials one launch evaluates
 */
int wkv_probe_ex2_rate(float *scratch_dev, int32_t blocks, int32_t threads, int32_t iters,
                       int64_t *ex2_per_launch, void *cuda_stream);

/*
 * Measurement aid (no counterpart in the paper): the rate of the cross-lane column sum a single-sweep
 * score kernel would need (a warp holds a 32 x 32 block of values, one row per lane, and sums its
 * columns over the lanes with 31 shuffle-and-add steps), in block elements per launch.  Compared with
 * wkv_probe_ex2_rate it tells whether replacing the second sweep's exponentials by such a reduction
 * could be faster.  Arguments as wkv_probe_ex2_rate.
 */
int wkv_probe_colsum_rate(float *scratch_dev, int32_t blocks, int32_t threads, int32_t iters,
                          int64_t *elements_per_launch, void *cuda_stream);

const char *wkv_status_string(int status);
const char *wkv_last_error_detail(void);
/* Number of kernels the library has launched from this process (all threads). */
uint64_t wkv_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* WKV_H_ */
