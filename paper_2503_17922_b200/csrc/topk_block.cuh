// Budgeted window selection (sentence after Eq. 4) for one unit by one thread block: the k-th
// largest window score is found with a 4-pass, 8-bit radix select over an order-preserving
// integer image of the fp32 scores, then the selected window indices are emitted in ascending
// order with block-wide prefix sums.  Equal scores at the threshold go to the lower window
// index.  Integer arithmetic only after the key mapping, so the result is exact and
// deterministic.  Used by the stand-alone selection kernel and by the fused score kernel.
#pragma once

#include "wkv_internal.cuh"

namespace wkv {

struct TopkSmem {
    int hist[256];
    int warp_sums[32];
    unsigned prefix;
    int remaining;
    int last_selected;
};

// larger float <=> larger key; -0 and +0 map to the same key
__device__ __forceinline__ unsigned topk_order_key(float f)
{
    unsigned u = __float_as_uint(f);
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// exclusive prefix sum of `v` over the NT threads of the block; also returns the total
template <int NT>
__device__ __forceinline__ int topk_block_scan(int v, int *warp_sums, int &total)
{
    constexpr int kWarps = NT / 32;
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

// All NT threads of the block call this.  `sc` are the unit's kw window scores (read through L2,
// so scores written by other blocks of the same grid are seen once the caller has synchronised
// with them), `out` receives k ascending indices followed by -1 up to k_max.
template <int NT>
__device__ void select_topk_block(TopkSmem &sm, const float *sc, int kw, int k, int k_max, int *out,
                                  int *kept_len_out, int n, int alpha, int omega)
{
    static_assert(NT % 32 == 0 && NT <= 1024, "block size");
    for (int x = (k > 0 ? k : 0) + threadIdx.x; x < k_max; x += NT) out[x] = -1;
    const int obs_rows = n < alpha ? n : alpha;
    if (k <= 0) {
        if (threadIdx.x == 0) *kept_len_out = obs_rows;
        return;
    }
    // ---- radix select: key of the k-th largest score --------------------------------
    if (threadIdx.x == 0) {
        sm.prefix = 0u;
        sm.remaining = k;
        sm.last_selected = 0;
    }
    unsigned mask = 0u;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int x = threadIdx.x; x < 256; x += NT) sm.hist[x] = 0;
        __syncthreads();
        const unsigned prefix = sm.prefix;
        const int remaining = sm.remaining;
        for (int w = threadIdx.x; w < kw; w += NT) {
            const unsigned key = topk_order_key(__ldcg(sc + w));
            if ((key & mask) == prefix) atomicAdd(&sm.hist[(key >> shift) & 0xffu], 1);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // warp 0: the bin (scanning from the top) in which the count reaches `remaining`
            const int lane = threadIdx.x;
            int c[8], tot = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                c[i] = sm.hist[lane * 8 + i];
                tot += c[i];
            }
            int incl = tot;   // inclusive suffix sum over the lanes (lane 31 holds the top bins)
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int t = __shfl_down_sync(0xffffffffu, incl, o);
                if (lane + o < 32) incl += t;
            }
            const int above = incl - tot;
            if (above < remaining && remaining <= incl) {
                int rem = remaining - above, bin = lane * 8;
#pragma unroll
                for (int i = 7; i >= 0; --i) {
                    if (c[i] >= rem) {
                        bin = lane * 8 + i;
                        break;
                    }
                    rem -= c[i];
                }
                sm.prefix = prefix | ((unsigned)bin << shift);
                sm.remaining = rem;   // after the last pass: how many keys equal to the threshold are taken
            }
        }
        mask |= 0xffu << shift;
        __syncthreads();
    }
    const unsigned thr = sm.prefix;
    const int need_eq = sm.remaining;

    // ---- ordered compaction ----------------------------------------------------------
    int eq_base = 0, out_base = 0;
    for (int w0 = 0; w0 < kw; w0 += NT) {
        const int w = w0 + threadIdx.x;
        unsigned key = 0u;
        const bool in = w < kw;
        if (in) key = topk_order_key(__ldcg(sc + w));
        const int is_eq = in && key == thr;
        int eq_total, sel_total;
        const int eq_rank = eq_base + topk_block_scan<NT>(is_eq, sm.warp_sums, eq_total);
        const int sel = in && (key > thr || (is_eq && eq_rank < need_eq));
        const int pos = out_base + topk_block_scan<NT>(sel, sm.warp_sums, sel_total);
        if (sel) {
            out[pos] = w;
            if (w == kw - 1) sm.last_selected = 1;
        }
        eq_base += eq_total;
        out_base += sel_total;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int n_r = n - alpha;
        const int last_size = n_r - (kw - 1) * omega;     // real size of the last window
        *kept_len_out = k * omega - (sm.last_selected ? omega - last_size : 0) + obs_rows;
    }
}

}  // namespace wkv
