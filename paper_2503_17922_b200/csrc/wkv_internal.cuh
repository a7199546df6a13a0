// Internal declarations shared by the library's translation units (host side of
// the C ABI and the kernel launchers).  Not part of the public interface.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <math.h>
#include <stdint.h>
#include <stddef.h>

#include "wkv.h"

namespace wkv {

// Shape as the kernels see it: plain values, device pointers only.
struct KShape {
    int batch, hq, hkv, d;
    int alpha, omega, p;       // p already resolved from task/top_p (Eq. 4)
    int max_seqlen, budget;
    int total_rows;            // sum of the sequence lengths (rows of the packed layout)
    int G, R;                  // query heads per KV head; observation rows per unit = G*alpha
    int kw_max, k_max, nr_max; // leading sizes of window_scores / window_idx / token_scores
    int n_cap;                 // no sequence is taken to be longer than this on the device:
                               // min(max_seqlen, alpha + kw_max * omega), so that a device copy of
                               // cu_seqlens that disagrees with the host copy cannot lead a kernel
                               // past the arrays that were sized from the host copy
    const int *cu;             // device cu_seqlens or nullptr
    const int *budgets;        // device budgets or nullptr
    long long sb, sh, st;      // K/V element strides
    long long qsb, qsh, qst;   // Q_obs element strides
    float scale_log2;          // log2(e)/sqrt(d): logits are handled in base 2
};

// Per-sequence integers, the same formulas on host and device (Eq. 3 and the
// budget sentence after Eq. 4).
__host__ __device__ inline int num_windows(int n, int alpha, int omega)
{
    return n <= alpha ? 0 : (n - alpha + omega - 1) / omega;
}
__host__ __device__ inline int num_selected(int n, int alpha, int omega, int budget)
{
    int kw = num_windows(n, alpha, omega);
    int k = budget > alpha ? (budget - alpha) / omega : 0;
    return k < kw ? k : kw;
}
// the same, never beyond the leading size of window_idx (device side: budgets_dev is not trusted further)
__host__ __device__ inline int num_selected_capped(int n, int alpha, int omega, int budget, int k_max)
{
    const int k = num_selected(n, alpha, omega, budget);
    return k < k_max ? k : k_max;
}

struct SeqInfo {
    int n;          // context length
    long long off;  // first row of the sequence in the packed layout (0 when dense)
    int budget;
};

__device__ inline SeqInfo seq_info(const KShape &s, int b)
{
    SeqInfo r;
    if (s.cu) {
        int lo = s.cu[b];
        r.n = s.cu[b + 1] - lo;
        // a device copy that disagrees with the host copy must not lead outside the packed tensor
        lo = lo < 0 ? 0 : (lo > s.total_rows ? s.total_rows : lo);
        r.n = r.n < 0 ? 0 : (r.n > s.n_cap ? s.n_cap : r.n);
        if (r.n > s.total_rows - lo) r.n = s.total_rows - lo;
        r.off = lo;
    } else {
        r.n = s.max_seqlen;
        r.off = 0;
    }
    r.budget = s.budgets ? s.budgets[b] : s.budget;
    return r;
}

// Workspace carve-up (all offsets 256-byte aligned).
struct Workspace {
    size_t status_off;   // int: device status word, only ever OR-ed by the kernels (0 = no error)
    size_t sync_off;     // int [kSyncTickets + kSyncWordsPerUnit * units], self-resetting
    size_t pstats_off;   // u64 [units][n_stat_chunks][128]: self-validating (max, sum) entries of the pipelined kernel;
                         // zero between launches (the kernel that writes them clears them again)
    size_t stats_off;    // float2 [units][n_stat_chunks][R_pad]  partial (max, sum) per row
    size_t lse_off;      // float  [units][R_pad]                 log2 of the row normaliser
    size_t scores_off;   // float  [units][kw_max]                window scores when the caller passes none
    size_t total;
    int n_stat_chunks;
    int r_pad;
};

// words of the synchronisation area before the per-unit words; unit u owns four words from
// sync[kSyncTickets + 4u]: ticket count, arrivals of the statistics sweep, "selection published" flag
// and gather job counter (the last two only in the kernel that also gathers)
constexpr int kSyncTickets = 16;
constexpr int kSyncWordsPerUnit = 4;

// per-device host state (kernel attributes, device properties) is kept for this many device ordinals
constexpr int kMaxDevices = 64;

constexpr int kStatChunk = 512;   // keys per partial-statistics chunk of the CUDA-core kernels

// Tensor-core kernels: key tiles of 128, at most 16 (+1 for window alignment) tiles per block, and a
// grid aimed at one wave of the 148 SMs of a B200 when the problem is small enough for that.
constexpr int kTcTileKeys = 128;
constexpr int kTcMaxChunkTiles = 16;
constexpr int kTcTargetBlocks = 148;
constexpr int kTcMaxWindow = 1024;

// The tensor-core kernel works through the units in waves whose keys fit the L2 cache together, so
// that the second sweep over a wave's keys is served from L2.  kTcWaveBytes is the budget.
constexpr long long kTcWaveBytes = 80ll << 20;

struct TcPlan {
    int units_per_wave;   // units swept together
    int chunks_per_unit;  // work items per unit
};
__host__ __device__ inline TcPlan tc_plan(int units, int max_seqlen, int head_dim)
{
    TcPlan p;
    const long long unit_bytes = (long long)max_seqlen * head_dim * 2;
    long long upw = kTcWaveBytes / (unit_bytes > 0 ? unit_bytes : 1);
    const int max_tiles = (max_seqlen + kTcTileKeys - 1) / kTcTileKeys;
    // A unit needs at least ceil(max_tiles / kTcMaxChunkTiles) blocks: no more units in a wave than
    // the SMs can take at that rate, or some blocks get two items of a wave and the others wait for
    // them.
    const int min_chunks = (max_tiles + kTcMaxChunkTiles - 1) / kTcMaxChunkTiles;
    if (upw > kTcTargetBlocks / min_chunks) upw = kTcTargetBlocks / min_chunks;
    if (upw < 1) upw = 1;
    if (upw > units) upw = units;
    p.units_per_wave = (int)upw;
    int a = kTcTargetBlocks / p.units_per_wave;
    const int b = (max_tiles + kTcMaxChunkTiles - 1) / kTcMaxChunkTiles;
    if (a < 1) a = 1;
    if (a > max_tiles) a = max_tiles;
    p.chunks_per_unit = a > b ? a : b;
    return p;
}
// The pipelined group kernel takes the units in waves too, but keeps TWO waves in flight (the
// statistics sweep runs one wave ahead of the scoring sweep), so two waves' keys share the L2 budget;
// with at least two units it always makes at least two waves, so that the gather of one wave's rows
// can run beside the scoring of the next.
struct PipePlan {
    int units_per_wave, chunks_per_unit, skew;
};
__host__ __device__ inline PipePlan pipe_plan(int units, int max_seqlen, int head_dim)
{
    PipePlan p;
    const long long unit_bytes = (long long)max_seqlen * head_dim * 2;
    const int max_tiles = (max_seqlen + kTcTileKeys - 1) / kTcTileKeys;
    const int min_chunks = (max_tiles + kTcMaxChunkTiles - 1) / kTcMaxChunkTiles;
    long long upw = (kTcWaveBytes / 2) / (unit_bytes > 0 ? unit_bytes : 1);
    if (upw > kTcTargetBlocks / min_chunks) upw = kTcTargetBlocks / min_chunks;
    if (upw > (units + 1) / 2) upw = (units + 1) / 2;
    if (upw < 1) upw = 1;
    p.units_per_wave = (int)upw;
    p.skew = units > p.units_per_wave ? 1 : 0;
    int a = kTcTargetBlocks / p.units_per_wave;
    if (a < 1) a = 1;
    if (a > max_tiles) a = max_tiles;
    p.chunks_per_unit = a > min_chunks ? a : min_chunks;
    return p;
}
// keys per block when `n_keys` keys are split over `chunks` blocks in whole tiles, rounded up to a
// multiple of `align` (1 for the statistics sweep, omega for the scoring sweep)
__host__ __device__ inline int tc_chunk_len(int n_keys, int chunks, int align)
{
    const int tiles = (n_keys + kTcTileKeys - 1) / kTcTileKeys;
    const int ct = (tiles + chunks - 1) / chunks;
    const int len = ct * kTcTileKeys;
    return (len + align - 1) / align * align;
}

// device status bits
constexpr int kStatusWaitExpired = 1;   // a bounded wait inside a kernel ran out; results are invalid

Workspace plan_workspace(const KShape &ks);

// Launchers (each returns a cudaError_t from the launch).
cudaError_t launch_score_simt(const KShape &ks, int dtype, const void *q, const void *k,
                              float *window_scores, float *token_scores,
                              void *workspace, const Workspace &ws, cudaStream_t stream,
                              const float *lse_obs = nullptr);
bool score_tc_supported(const KShape &ks, int dtype);
// window_idx / kept_len non-null: the selection is fused into the same launch.
// lse_obs non-null: float [B, H_q, alpha], natural log of Eq. 1's normaliser of every observation
// row, supplied by the caller; the statistics sweep is then skipped.
int launch_score_tc(const KShape &ks, const void *q, const void *k,
                    float *window_scores, float *token_scores, int *window_idx, int *kept_len,
                    void *workspace, const Workspace &ws, cudaStream_t stream, const float *lse_obs = nullptr);
// The pipelined group kernel (score_pipe.cu): scoring, selection and, with `gather`, the shared-index
// gather of every layer in one launch.  R <= 128 only.
struct LayerTable;
struct PipeGather {
    int n_tensors;
    const LayerTable *tab;
    const int *cu_out;
    int keep_capacity;
};
bool group_pipeline_supported(const KShape &ks, int dtype);
bool group_pipeline_can_gather(const KShape &ks, int elem_bytes, int n_tensors);
int launch_group_pipeline(const KShape &ks, const void *q, const void *k, float *window_scores, float *token_scores,
                          int *window_idx, int *kept_len, void *workspace, const Workspace &ws, cudaStream_t stream,
                          const float *lse_obs, const PipeGather *gather);
cudaError_t launch_topk(const KShape &ks, const float *window_scores, int *window_idx, int *kept_len,
                        cudaStream_t stream);

struct LayerTable {
    const void *src[2 * WKV_MAX_GROUP_LAYERS];
    void *dst[2 * WKV_MAX_GROUP_LAYERS];
};
// paged compact cache: strides of the page pool in elements
struct PagedOut {
    const int *block_table;   // device [batch][max_pages]
    int max_pages, page_size, num_pages;
    long long page_stride, head_stride, row_stride;
};
cudaError_t launch_gather(const KShape &ks, int elem_bytes, int n_tensors, const LayerTable &tab,
                          const int *window_idx, const int *cu_out, int keep_capacity,
                          cudaStream_t stream, const PagedOut *paged = nullptr);
// compaction of every layer's K/V inside its own buffer (compact.cu)
struct InplaceTable {
    void *ptr[2 * WKV_MAX_GROUP_LAYERS];
};
cudaError_t launch_compact_inplace(const KShape &ks, int elem_bytes, int n_tensors, const InplaceTable &tab,
                                   const int *window_idx, cudaStream_t stream);

// Eq. 4 for one window of `size` values: mean of the p largest.  Elements are visited in the
// strict order (value descending, position ascending), so equal values are each taken once.
__device__ inline float pool_top_p(const float *w, int size, int p)
{
    if (p >= size) {
        float acc = 0.f;
        for (int x = 0; x < size; ++x) acc += w[x];
        return acc / (float)size;
    }
    float acc = 0.f, prev_v = INFINITY;
    int prev_i = -1;
    for (int round = 0; round < p; ++round) {
        float best_v = -INFINITY;
        int best_i = size;
        for (int x = 0; x < size; ++x) {
            float v = w[x];
            bool after_prev = v < prev_v || (v == prev_v && x > prev_i);
            if (after_prev && (v > best_v || best_i == size)) {
                best_v = v;
                best_i = x;
            }
        }
        acc += best_v;
        prev_v = best_v;
        prev_i = best_i;
    }
    return acc / (float)p;
}

// host side of the boundary, shared by the translation units that export entry points
int resolve(const wkv_shape *s, KShape &ks);            // validates the shape, fills the kernel-side copy
int check_cuda(cudaError_t e, const char *what);         // cudaError_t -> wkv_status with detail
// scoring; with window_idx / kept_len non-null also the selection (one launch on the tensor-core path)
// `gather` non-null: the caller wants the layers gathered as well; *gathered tells whether the launch
// that scored has done it (else the caller launches the gather kernel)
int do_score(const wkv_shape *s, const KShape &ks, const Workspace &ws, const void *q, const void *k,
             float *window_scores, float *token_scores, int *window_idx, int *kept_len, void *workspace,
             cudaStream_t stream, const float *lse_obs = nullptr, const PipeGather *gather = nullptr,
             bool *gathered = nullptr);

void count_launches(int n);
uint64_t launches_so_far();
// the group call behind wkv_compress_group / wkv_compress_group_lse (lse_obs may be null)
int compress_group_entry(const wkv_shape *s, int32_t n_layers, const void *q_obs_leader, const float *lse_obs,
                         const void *const *k_layers, const void *const *v_layers, void *const *k_out_layers,
                         void *const *v_out_layers, float *window_scores, int32_t *window_idx, int32_t *kept_len,
                         const int32_t *cu_seqlens_out, int32_t keep_capacity, void *workspace,
                         size_t workspace_bytes, void *cuda_stream);
void set_error_detail(const char *fmt, ...);

}  // namespace wkv
