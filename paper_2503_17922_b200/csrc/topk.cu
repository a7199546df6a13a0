// Budgeted window selection (sentence after Eq. 4): one thread block per unit finds
// the k-th largest window score with a 4-pass, 8-bit radix select over an
// order-preserving integer image of the fp32 scores, then emits the selected window
// indices in ascending order with block-wide prefix sums.  Equal scores at the
// threshold go to the lower window index.  Integer arithmetic only after the key
// mapping, so the result is exact and deterministic.
#include "wkv_internal.cuh"

namespace wkv {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;

// larger float <=> larger key; -0 and +0 map to the same key
__device__ inline unsigned order_key(float f)
{
    unsigned u = __float_as_uint(f);
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// exclusive prefix sum of `v` over the block (blockDim = kThreads); also returns the total
__device__ inline int block_exclusive_scan(int v, int *warp_sums, int &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();   // protects warp_sums from the previous use
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        int x = warp_sums[w];
        if (w < warp) base += x;
        tot += x;
    }
    total = tot;
    return base + incl - v;
}

__global__ void __launch_bounds__(kThreads)
select_topk_kernel(KShape s, const float *__restrict__ window_scores, int *__restrict__ window_idx,
                   int *__restrict__ kept_len)
{
    __shared__ int hist[256];
    __shared__ int warp_sums[kWarps];
    __shared__ unsigned sh_prefix;
    __shared__ int sh_remaining;
    __shared__ int sh_last_selected;

    const int unit = blockIdx.x;
    const int b = unit / s.hkv;
    const SeqInfo si = seq_info(s, b);
    const int n = si.n;
    const int kw = num_windows(n, s.alpha, s.omega);
    const int k = num_selected(n, s.alpha, s.omega, si.budget);
    const float *sc = window_scores + (size_t)unit * s.kw_max;
    int *out = window_idx + (size_t)unit * s.k_max;

    for (int x = k + threadIdx.x; x < s.k_max; x += kThreads) out[x] = -1;
    const int obs_rows = n < s.alpha ? n : s.alpha;
    if (k <= 0) {
        if (threadIdx.x == 0) kept_len[unit] = obs_rows;
        return;
    }

    // ---- radix select: key of the k-th largest score --------------------------------
    if (threadIdx.x == 0) {
        sh_prefix = 0u;
        sh_remaining = k;
        sh_last_selected = 0;
    }
    unsigned mask = 0u;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int x = threadIdx.x; x < 256; x += kThreads) hist[x] = 0;
        __syncthreads();
        const unsigned prefix = sh_prefix;
        for (int w = threadIdx.x; w < kw; w += kThreads) {
            unsigned key = order_key(sc[w]);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 0xffu], 1);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int remaining = sh_remaining, bin = 255;
            for (; bin > 0; --bin) {
                int c = hist[bin];
                if (c >= remaining) break;
                remaining -= c;
            }
            sh_prefix = prefix | ((unsigned)bin << shift);
            sh_remaining = remaining;   // how many keys equal to the final threshold are taken
        }
        mask |= 0xffu << shift;
        __syncthreads();
    }
    const unsigned thr = sh_prefix;
    const int need_eq = sh_remaining;

    // ---- ordered compaction ----------------------------------------------------------
    int eq_base = 0, out_base = 0;
    for (int w0 = 0; w0 < kw; w0 += kThreads) {
        const int w = w0 + threadIdx.x;
        unsigned key = 0u;
        bool in = w < kw;
        if (in) key = order_key(sc[w]);
        const int is_eq = in && key == thr;
        int eq_total, sel_total;
        const int eq_rank = eq_base + block_exclusive_scan(is_eq, warp_sums, eq_total);
        const int sel = in && (key > thr || (is_eq && eq_rank < need_eq));
        const int pos = out_base + block_exclusive_scan(sel, warp_sums, sel_total);
        if (sel) {
            out[pos] = w;
            if (w == kw - 1) sh_last_selected = 1;
        }
        eq_base += eq_total;
        out_base += sel_total;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int n_r = n - s.alpha;
        const int last_size = n_r - (kw - 1) * s.omega;     // real size of the last window
        kept_len[unit] = k * s.omega - (sh_last_selected ? s.omega - last_size : 0) + obs_rows;
    }
}

}  // namespace

cudaError_t launch_topk(const KShape &ks, const float *window_scores, int *window_idx, int *kept_len,
                        cudaStream_t stream)
{
    const int units = ks.batch * ks.hkv;
    select_topk_kernel<<<units, kThreads, 0, stream>>>(ks, window_scores, window_idx, kept_len);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace wkv
