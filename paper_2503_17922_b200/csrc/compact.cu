// In-place compaction (section 2.2.2 during prefill: the compact cache of a layer takes the place of
// the layer's full K/V inside the buffer the prefill wrote them to).  The retained rows of a unit move
// to the front of the unit's own rows: output row r comes from source row src(r) >= r (window indices
// ascend, and the observation rows are the last rows of the sequence), so rows only ever move toward
// lower addresses.
//
// A parallel copy can still destroy a source row before it has been read: output window w lies on
// source window w, which an earlier output slot may need.  The kernel therefore gives one thread block
// a whole (unit, tensor) and lets it walk the output rows in ascending batches: all source rows of a
// batch are read into registers, the block synchronises, then the batch is written.  Inside a batch
// every read precedes every write; a later batch reads only rows at or behind its own output rows,
// which lie behind everything written so far.  Blocks never touch each other's units.
#include "wkv_internal.cuh"

namespace wkv {
namespace {

constexpr int kThreads = 1024;
constexpr int kVecs = 8;              // 16-byte vectors per thread and batch: 128 KB per block in flight

struct CompactParams {
    KShape s;
    InplaceTable tab;
    const int *window_idx;
    int vec_per_row;
    int elem_bytes;
};

__global__ void __launch_bounds__(kThreads, 1)
compact_inplace_kernel(const __grid_constant__ CompactParams prm)
{
    const KShape &s = prm.s;
    const int unit = blockIdx.x, tensor = blockIdx.y;
    const int b = unit / s.hkv, h = unit % s.hkv;
    const SeqInfo si = seq_info(s, b);
    const int n = si.n;
    const int n_r = n > s.alpha ? n - s.alpha : 0;
    const int kw = num_windows(n, s.alpha, s.omega);
    const int k = num_selected_capped(n, s.alpha, s.omega, si.budget, s.k_max);
    const int *idx = prm.window_idx + (size_t)unit * s.k_max;
    int review_rows = k * s.omega;
    if (k > 0 && idx[k - 1] == kw - 1) review_rows -= kw * s.omega - n_r;
    const int kept = review_rows + (n - n_r);

    const int vpr = prm.vec_per_row;
    const long long row_vecs = s.st * prm.elem_bytes / 16;
    int4 *base = reinterpret_cast<int4 *>(static_cast<char *>(prm.tab.ptr[tensor]) +
                                          (si.off * s.st + b * s.sb + h * s.sh) * (long long)prm.elem_bytes);
    const int rows_per_batch = max(1, (kThreads * kVecs) / vpr);
    for (int r0 = 0; r0 < kept; r0 += rows_per_batch) {
        const int rows = min(rows_per_batch, kept - r0);
        const int n_vec = rows * vpr;
        int4 val[kVecs];
        long long doff[kVecs];
#pragma unroll
        for (int u = 0; u < kVecs; ++u) {
            const int v = (int)threadIdx.x + u * kThreads;
            doff[u] = -1;
            if (v < n_vec) {
                const int r = r0 + v / vpr, c = v % vpr;
                int src_row;
                if (r < review_rows) {
                    const int wi = idx[r / s.omega];
                    // an entry that is no window of this sequence, or that lies before its own slot (a
                    // list that is not an ascending selection), is skipped: the row stays as it is
                    src_row = (wi < r / s.omega || wi >= kw) ? -1 : wi * s.omega + r % s.omega;
                } else {
                    src_row = n_r + (r - review_rows);
                }
                if (src_row >= 0 && src_row < n && src_row != r) {
                    val[u] = base[(long long)src_row * row_vecs + c];
                    doff[u] = (long long)r * row_vecs + c;
                }
            }
        }
        __syncthreads();      // every source row of the batch has been read
#pragma unroll
        for (int u = 0; u < kVecs; ++u)
            if (doff[u] >= 0) base[doff[u]] = val[u];
        __syncthreads();      // keeps the block in step: the next batch is read after this one is written
    }
}

}  // namespace

cudaError_t launch_compact_inplace(const KShape &ks, int elem_bytes, int n_tensors, const InplaceTable &tab,
                                   const int *window_idx, cudaStream_t stream)
{
    CompactParams prm;
    prm.s = ks;
    prm.tab = tab;
    prm.window_idx = window_idx;
    prm.vec_per_row = ks.d * elem_bytes / 16;
    prm.elem_bytes = elem_bytes;
    dim3 grid(ks.batch * ks.hkv, n_tensors);
    compact_inplace_kernel<<<grid, kThreads, 0, stream>>>(prm);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace wkv
