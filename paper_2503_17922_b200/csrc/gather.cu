// Shared-index gather (section 2.2.2): copies, for every layer tensor of the group,
// the rows of the selected review windows followed by the observation rows into
// the compact cache.  Pure bit copy with 16-byte vector accesses; a row of d
// elements is d*elem_bytes/16 vectors, consecutive threads take consecutive
// vectors so both the reads (omega consecutive rows per window) and the writes
// (consecutive output rows) are fully coalesced.
#include "wkv_internal.cuh"

namespace wkv {
namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;            // independent 16-byte loads in flight per thread

struct GatherParams {
    KShape s;
    LayerTable tab;
    const int *window_idx;
    const int *cu_out;
    int keep_capacity;
    int vec_per_row;                  // 16-byte vectors per row
    int elem_bytes;
    int rows_per_block;               // output rows handled by one block
};

__device__ inline int4 ld_stream(const int4 *p)
{
    int4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ inline void st_stream(int4 *p, const int4 &v)
{
    asm volatile("st.global.L1::no_allocate.v4.s32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y),
                 "r"(v.z), "r"(v.w)
                 : "memory");
}

__global__ void __launch_bounds__(kThreads)
gather_kv_kernel(const __grid_constant__ GatherParams prm)
{
    const KShape &s = prm.s;
    const int unit = blockIdx.y, tensor = blockIdx.z;
    const int b = unit / s.hkv, h = unit % s.hkv;
    const SeqInfo si = seq_info(s, b);
    const int n = si.n;
    const int n_r = n > s.alpha ? n - s.alpha : 0;
    const int kw = num_windows(n, s.alpha, s.omega);
    const int k = num_selected(n, s.alpha, s.omega, si.budget);
    const int *idx = prm.window_idx + (size_t)unit * s.k_max;

    // rows of the unit: the selected windows (only the last window of the sequence can be
    // short, and it can only be the last selected one), then the observation rows
    int review_rows = k * s.omega;
    if (k > 0 && idx[k - 1] == kw - 1) review_rows -= kw * s.omega - n_r;
    const int total_rows = review_rows + (n - n_r);

    const int row_begin = blockIdx.x * prm.rows_per_block;
    if (row_begin >= total_rows) return;
    const int row_end = min(total_rows, row_begin + prm.rows_per_block);

    const int vpr = prm.vec_per_row;
    // strides are multiples of 16 bytes (checked on the host), so vector indexing is exact
    const long long src_row_vecs = s.st * prm.elem_bytes / 16;    // vectors between consecutive source rows
    const int4 *src = reinterpret_cast<const int4 *>(
        static_cast<const char *>(prm.tab.src[tensor]) +
        (si.off * s.st + b * s.sb + h * s.sh) * (long long)prm.elem_bytes);
    int4 *dst;
    long long dst_row_vecs;
    if (prm.cu_out) {
        dst = reinterpret_cast<int4 *>(prm.tab.dst[tensor]) +
              ((long long)prm.cu_out[b] * s.hkv + h) * vpr;
        dst_row_vecs = (long long)s.hkv * vpr;
    } else {
        dst = reinterpret_cast<int4 *>(prm.tab.dst[tensor]) + (long long)unit * prm.keep_capacity * vpr;
        dst_row_vecs = vpr;
    }

    const int n_vec = (row_end - row_begin) * vpr;
    for (int v0 = threadIdx.x; v0 < n_vec; v0 += kThreads * kUnroll) {
        int4 val[kUnroll];
        long long doff[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int v = v0 + u * kThreads;
            if (v < n_vec) {
                const int r = row_begin + v / vpr, c = v % vpr;
                int src_row;
                if (r < review_rows) {
                    const int w = r / s.omega;
                    src_row = idx[w] * s.omega + (r - w * s.omega);
                } else {
                    src_row = n_r + (r - review_rows);
                }
                val[u] = ld_stream(src + src_row * src_row_vecs + c);
                doff[u] = r * dst_row_vecs + c;
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int v = v0 + u * kThreads;
            if (v < n_vec) st_stream(dst + doff[u], val[u]);
        }
    }
}

}  // namespace

cudaError_t launch_gather(const KShape &ks, int elem_bytes, int n_tensors, const LayerTable &tab,
                          const int *window_idx, const int *cu_out, int keep_capacity,
                          cudaStream_t stream)
{
    GatherParams prm;
    prm.s = ks;
    prm.tab = tab;
    prm.window_idx = window_idx;
    prm.cu_out = cu_out;
    prm.keep_capacity = keep_capacity;
    prm.vec_per_row = ks.d * elem_bytes / 16;
    prm.elem_bytes = elem_bytes;
    // each block moves about 64 KB so that a full-size group yields several waves of blocks
    int rows = (64 * 1024) / (prm.vec_per_row * 16);
    if (rows < 1) rows = 1;
    prm.rows_per_block = rows;
    // upper bound of rows per unit: all selected windows full + observation rows
    const int max_rows = ks.k_max * ks.omega + ks.alpha;
    dim3 grid((max_rows + rows - 1) / rows, ks.batch * ks.hkv, n_tensors);
    gather_kv_kernel<<<grid, kThreads, 0, stream>>>(prm);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace wkv
