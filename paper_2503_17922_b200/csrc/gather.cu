// Shared-index gather (section 2.2.2): copies, for every layer tensor of the group, the rows of
// the selected review windows followed by the observation rows into the compact cache.  Pure bit
// copy with 16-byte vector accesses.
//
// The unit of work is one window (omega consecutive source rows = omega consecutive output rows)
// of one unit of one tensor, taken by one warp: all its loads are issued before the first store
// (up to 8 x 16 bytes in flight per lane), and the index arithmetic is done once per window, not
// once per vector.  The observation rows are handled as extra windows behind the selected ones.
#include "wkv_internal.cuh"

namespace wkv {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kBatch = 8;             // independent 16-byte loads in flight per lane

struct GatherParams {
    KShape s;
    LayerTable tab;
    const int *window_idx;
    const int *cu_out;
    int keep_capacity;
    int vec_per_row;                  // 16-byte vectors per row
    int vec_shift;                    // log2(vec_per_row) when it is a power of two, else -1
    int elem_bytes;
    int slots_per_block;              // windows (selected + observation) handled by one block
    int obs_slots;                    // ceil(alpha / omega)
    // paged output (page_size > 0): row r of unit (b, h) lives in page block_table[b][r / page_size]
    const int *block_table;           // [batch][max_pages]
    int max_pages, page_size, num_pages;
    long long page_vecs, head_vecs, row_vecs;   // strides of the page pool in 16-byte vectors
};

__device__ __forceinline__ int4 ld_stream(const int4 *p)
{
    int4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(int4 *p, const int4 &v)
{
    asm volatile("st.global.L1::no_allocate.v4.s32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y),
                 "r"(v.z), "r"(v.w)
                 : "memory");
}

// PAGED is a separate instantiation: its per-row page arithmetic would otherwise cost the plain copy
// registers it needs for its loads in flight.
template <bool PAGED>
__global__ void __launch_bounds__(kThreads, 4)
gather_kv_kernel(const __grid_constant__ GatherParams prm)
{
    const KShape &s = prm.s;
    const int unit = blockIdx.y, tensor = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = unit / s.hkv, h = unit % s.hkv;
    const SeqInfo si = seq_info(s, b);
    const int n = si.n;
    const int n_r = n > s.alpha ? n - s.alpha : 0;
    const int kw = num_windows(n, s.alpha, s.omega);
    const int k = num_selected_capped(n, s.alpha, s.omega, si.budget, s.k_max);
    const int *idx = prm.window_idx + (size_t)unit * s.k_max;

    // rows of the unit: the selected windows (only the last window of the sequence can be short,
    // and it can only be the last selected one), then the observation rows
    int review_rows = k * s.omega;
    if (k > 0 && idx[k - 1] == kw - 1) review_rows -= kw * s.omega - n_r;
    const int obs_rows = n - n_r;

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
    constexpr bool paged = PAGED;
    const bool src_dense = src_row_vecs == vpr, dst_dense = dst_row_vecs == vpr && !paged;
    const int *pages = paged ? prm.block_table + (size_t)b * prm.max_pages : nullptr;
    if (paged) dst = reinterpret_cast<int4 *>(prm.tab.dst[tensor]) + (long long)h * prm.head_vecs;

    const int slot_end = min(k + prm.obs_slots, (int)(blockIdx.x + 1) * prm.slots_per_block);
    for (int slot = blockIdx.x * prm.slots_per_block + warp; slot < slot_end; slot += kWarps) {
        int src_row0, dst_row0, n_rows;
        if (slot < k) {
            // an entry that is no window of this sequence (a list that no selection has written, or
            // that the caller filled wrongly) is skipped: the kernel never leaves the tensors
            const int wi = idx[slot];
            if (wi < 0 || wi >= kw) continue;
            src_row0 = wi * s.omega;
            n_rows = min(s.omega, n_r - src_row0);
            dst_row0 = slot * s.omega;
        } else {
            const int o = (slot - k) * s.omega;
            src_row0 = n_r + o;
            n_rows = min(s.omega, obs_rows - o);
            dst_row0 = review_rows + o;
        }
        if (n_rows <= 0) continue;
        // dense output: a unit owns keep_capacity rows (cannot trigger while the device copies of
        // cu_seqlens / budgets equal the host copies the capacity was checked against)
        if (!prm.cu_out && !paged && dst_row0 + n_rows > prm.keep_capacity) continue;
        if (paged) {
            // every row finds its page; a row whose page entry is missing or negative is skipped
            const int n_vec = n_rows * vpr;
            for (int v0 = lane; v0 < n_vec; v0 += 32 * kBatch) {
                int4 val[kBatch];
                long long doff[kBatch];
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int v = v0 + u * 32;
                    doff[u] = -1;
                    if (v < n_vec) {
                        const int r = prm.vec_shift >= 0 ? v >> prm.vec_shift : v / vpr;
                        const int c = v - r * vpr;
                        const int row = dst_row0 + r, page = row / prm.page_size;
                        const int phys = page < prm.max_pages ? pages[page] : -1;
                        if (phys >= 0 && phys < prm.num_pages)
                            doff[u] = (long long)phys * prm.page_vecs + (long long)(row - page * prm.page_size) * prm.row_vecs + c;
                        val[u] = ld_stream(src + (long long)(src_row0 + r) * src_row_vecs + c);
                    }
                }
#pragma unroll
                for (int u = 0; u < kBatch; ++u)
                    if (doff[u] >= 0) st_stream(dst + doff[u], val[u]);
            }
            continue;
        }
        const int4 *sp = src + src_row0 * src_row_vecs;
        int4 *dp = dst + dst_row0 * dst_row_vecs;
        const int n_vec = n_rows * vpr;
        for (int v0 = lane; v0 < n_vec; v0 += 32 * kBatch) {
            int4 val[kBatch];
            int soff[kBatch], doff[kBatch];   // offsets inside one window: small
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int v = v0 + u * 32;
                if (v < n_vec) {
                    soff[u] = v;
                    doff[u] = v;
                    if (!src_dense || !dst_dense) {
                        const int r = prm.vec_shift >= 0 ? v >> prm.vec_shift : v / vpr;
                        const int c = v - r * vpr;
                        if (!src_dense) soff[u] = r * (int)src_row_vecs + c;
                        if (!dst_dense) doff[u] = r * (int)dst_row_vecs + c;
                    }
                    val[u] = ld_stream(sp + soff[u]);
                }
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
                if (v0 + u * 32 < n_vec) st_stream(dp + doff[u], val[u]);
        }
    }
}

}  // namespace

cudaError_t launch_gather(const KShape &ks, int elem_bytes, int n_tensors, const LayerTable &tab,
                          const int *window_idx, const int *cu_out, int keep_capacity,
                          cudaStream_t stream, const PagedOut *paged)
{
    GatherParams prm;
    prm.block_table = nullptr;
    prm.max_pages = prm.page_size = prm.num_pages = 0;
    prm.page_vecs = prm.head_vecs = prm.row_vecs = 0;
    if (paged) {
        prm.block_table = paged->block_table;
        prm.max_pages = paged->max_pages;
        prm.page_size = paged->page_size;
        prm.num_pages = paged->num_pages;
        prm.page_vecs = paged->page_stride * elem_bytes / 16;
        prm.head_vecs = paged->head_stride * elem_bytes / 16;
        prm.row_vecs = paged->row_stride * elem_bytes / 16;
    }
    prm.s = ks;
    prm.tab = tab;
    prm.window_idx = window_idx;
    prm.cu_out = cu_out;
    prm.keep_capacity = keep_capacity;
    prm.vec_per_row = ks.d * elem_bytes / 16;
    prm.vec_shift = -1;
    for (int sh = 0; sh < 16; ++sh)
        if ((1 << sh) == prm.vec_per_row) prm.vec_shift = sh;
    prm.elem_bytes = elem_bytes;
    prm.obs_slots = (ks.alpha + ks.omega - 1) / ks.omega;
    // each warp moves a few windows; a block takes about 64 KB
    const long long window_bytes = (long long)ks.omega * prm.vec_per_row * 16;
    long long per_block = (64 * 1024) / window_bytes;
    if (per_block < kWarps) per_block = kWarps;
    prm.slots_per_block = (int)per_block;
    const int max_slots = ks.k_max + prm.obs_slots;
    dim3 grid((max_slots + prm.slots_per_block - 1) / prm.slots_per_block, ks.batch * ks.hkv, n_tensors);
    if (paged) gather_kv_kernel<true><<<grid, kThreads, 0, stream>>>(prm);
    else gather_kv_kernel<false><<<grid, kThreads, 0, stream>>>(prm);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace wkv
