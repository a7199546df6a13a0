// Budgeted window selection (sentence after Eq. 4) for one unit by one thread block: the k-th
// largest window score is found with a radix select (11 bits per pass, only over the bits in which
// the unit's keys differ, finished by direct ranking once few candidates are left) over an
// order-preserving integer image of the fp32 scores, then the selected window indices are emitted
// in ascending order with one block-wide prefix sum.  Equal scores at the threshold go to the
// lower window index.  Integer arithmetic only after the key mapping, so the result is exact and
// deterministic.  Used by the stand-alone selection kernel and by the fused score kernel.
#pragma once

#include "wkv_internal.cuh"

namespace wkv {

constexpr int kTopkBins = 2048;

struct TopkSmem {
    __align__(16) int hist[kTopkBins];
    int warp_sums[33];
    unsigned prefix;
    int remaining;
    int last_selected;
    unsigned kmin, kmax;        // smallest and largest key of the unit
    int cand_total, n_cand;     // keys in the chosen bin; candidates collected for the direct finish
    unsigned cand[64];
};
constexpr int kTopkDirect = 64;  // with at most this many candidates left, rank them directly

// larger float <=> larger key; -0 and +0 map to the same key
__device__ __forceinline__ unsigned topk_order_key(float f)
{
    unsigned u = __float_as_uint(f);
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// exclusive prefix sum of `v` over the NT threads of the block; also returns the total.  Shared
// memory is one pipe for the whole SM, so the scan touches it as little as possible: one word
// written per warp, the warp totals scanned by warp 0 with shuffles, two words read per thread.
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
    if (warp == 0) {
        const int mine = lane < kWarps ? warp_sums[lane] : 0;
        int w_incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, w_incl, o);
            if (lane >= o) w_incl += t;
        }
        if (lane < kWarps) warp_sums[lane] = w_incl - mine;       // exclusive base of warp `lane`
        if (lane == 31) warp_sums[32] = w_incl;                    // grand total
    }
    __syncthreads();
    total = warp_sums[32];
    return warp_sums[warp] + incl - v;
}

// All NT threads of the block call this.  `sc` are the unit's kw window scores (read through L2,
// so scores written by other blocks of the same grid are seen once the caller has synchronised
// with them), `out` receives k ascending indices followed by -1 up to k_max.
// Thread t owns the windows [t*E, (t+1)*E), E = ceil(kw / NT).  With E <= REGS (4 or 8) the keys
// are read once and stay in registers through the radix passes and the compaction (one trip to L2
// instead of five); REGS = 0: longer lists are re-read.
template <int NT, int REGS>
__device__ __forceinline__ void select_topk_impl(TopkSmem &sm, const float *sc, int kw, int k, int *out,
                                                 int *kept_len_out, int n, int alpha, int omega, int obs_rows)
{
    // the histogram is scanned by `kScanners` threads (a power of two), kBinsPer bins each
    constexpr int kScanners = NT >= 512 ? 512 : 256;
    constexpr int kBinsPer = kTopkBins / kScanners;
    static_assert(NT >= 256, "block size");
    const int E = (kw + NT - 1) / NT;
    const int w_lo = min(kw, (int)threadIdx.x * E), w_hi = min(kw, w_lo + E);
    constexpr bool IN_REGS = REGS > 0;
    constexpr int kTopkRegs = IN_REGS ? REGS : 1;
    unsigned keys[kTopkRegs];
    if (IN_REGS) {
#pragma unroll
        for (int e = 0; e < kTopkRegs; ++e) keys[e] = w_lo + e < w_hi ? topk_order_key(__ldcg(sc + w_lo + e)) : 0u;
    }
    auto key_at = [&](int e) -> unsigned { return IN_REGS ? keys[e] : topk_order_key(__ldcg(sc + w_lo + e)); };

    // ---- radix select: key of the k-th largest score --------------------------------
    // Keys are taken relative to the smallest one, and only the bits in which the largest differs
    // from it are resolved, 11 at a time from the top (window scores share sign and most of the
    // exponent: typically one pass), until at most kTopkDirect candidates share the prefix; those
    // are ranked against each other directly.
    if (threadIdx.x == 0) {
        sm.prefix = 0u;
        sm.remaining = k;
        sm.last_selected = 0;
        sm.kmin = 0xffffffffu;
        sm.kmax = 0u;
        sm.cand_total = kw;
        sm.n_cand = 0;
    }
    for (int x = threadIdx.x; x < kTopkBins; x += NT) sm.hist[x] = 0;
    __syncthreads();
    {
        unsigned lo = 0xffffffffu, hi = 0u;
        if (IN_REGS) {
#pragma unroll
            for (int e = 0; e < kTopkRegs; ++e)
                if (w_lo + e < w_hi) {
                    lo = min(lo, keys[e]);
                    hi = max(hi, keys[e]);
                }
        } else {
            for (int e = 0; w_lo + e < w_hi; ++e) {
                const unsigned key = key_at(e);
                lo = min(lo, key);
                hi = max(hi, key);
            }
        }
        lo = __reduce_min_sync(0xffffffffu, lo);
        hi = __reduce_max_sync(0xffffffffu, hi);
        if ((threadIdx.x & 31) == 0) {
            atomicMin(&sm.kmin, lo);
            atomicMax(&sm.kmax, hi);
        }
    }
    __syncthreads();
    const unsigned kmin = sm.kmin;
    const int bits = 32 - __clz(sm.kmax - kmin);     // 0 when all keys are equal
    unsigned mask = 0u;
    int top = bits;                                   // bits [top, 32) of (key - kmin) are resolved
#pragma unroll 1
    while (top > 0) {
        const unsigned prefix = sm.prefix;
        const int remaining = sm.remaining;
        if (sm.cand_total <= kTopkDirect) {
            // direct finish: collect the candidates, rank each against the others
#pragma unroll
            for (int e = 0; e < (IN_REGS ? kTopkRegs : E); ++e) {
                if (IN_REGS && e >= E) break;
                if (w_lo + e < w_hi) {
                    const unsigned rk = key_at(e) - kmin;
                    if ((rk & mask) == prefix) sm.cand[atomicAdd(&sm.n_cand, 1)] = rk;
                }
            }
            __syncthreads();
            const int n_cand = sm.n_cand;
            if ((int)threadIdx.x < n_cand) {
                const unsigned my = sm.cand[threadIdx.x];
                int gt = 0, eq = 0;
                for (int j = 0; j < n_cand; ++j) {
                    const unsigned o = sm.cand[j];
                    gt += o > my;
                    eq += o == my;
                }
                if (gt < remaining && remaining <= gt + eq) {   // every thread that gets here writes the same values
                    sm.prefix = my;
                    sm.remaining = remaining - gt;
                }
            }
            __syncthreads();
            break;
        }
        const int low = top > 11 ? top - 11 : 0;
        const unsigned digit_mask = (1u << (top - low)) - 1u;
#pragma unroll
        for (int e = 0; e < (IN_REGS ? kTopkRegs : E); ++e) {
            if (IN_REGS && e >= E) break;   // uniform: E is the same for every thread
            unsigned bin = kTopkBins;       // not taking part in this pass
            if (w_lo + e < w_hi) {
                const unsigned rk = key_at(e) - kmin;
                if ((rk & mask) == prefix) bin = (rk >> low) & digit_mask;
            }
            // the lanes that share the bin of the first participating lane are counted by that lane
            const unsigned part = __ballot_sync(0xffffffffu, bin < kTopkBins);
            if (part) {
                const int leader = __ffs(part) - 1;
                const unsigned pivot = __shfl_sync(0xffffffffu, bin, leader);
                const unsigned same = __ballot_sync(0xffffffffu, bin == pivot);
                if ((int)(threadIdx.x & 31) == leader) atomicAdd(&sm.hist[pivot], __popc(same));
                else if (bin < kTopkBins && bin != pivot) atomicAdd(&sm.hist[bin], 1);
            }
        }
        __syncthreads();
        // the bin (scanning from the top) in which the count reaches `remaining`
        int c[kBinsPer], mine = 0;
        if (threadIdx.x < kScanners) {
            int4 *hv = reinterpret_cast<int4 *>(sm.hist + threadIdx.x * kBinsPer);
#pragma unroll
            for (int i = 0; i < kBinsPer; i += 4) {
                const int4 x = hv[i / 4];
                hv[i / 4] = make_int4(0, 0, 0, 0);   // ready for the next pass
                c[i] = x.x;
                c[i + 1] = x.y;
                c[i + 2] = x.z;
                c[i + 3] = x.w;
                mine += (x.x + x.y) + (x.z + x.w);
            }
        }
        int total;
        const int below = topk_block_scan<NT>(mine, sm.warp_sums, total);   // keys in lower bins
        const int above = total - below - mine;
        if (threadIdx.x < kScanners && above < remaining && remaining <= above + mine) {
            int rem = remaining - above, bin = threadIdx.x * kBinsPer;
#pragma unroll
            for (int i = kBinsPer - 1; i >= 0; --i) {
                if (c[i] >= rem) {
                    bin = threadIdx.x * kBinsPer + i;
                    sm.cand_total = c[i];
                    break;
                }
                rem -= c[i];
            }
            sm.prefix = prefix | ((unsigned)bin << low);
            sm.remaining = rem;   // after the last pass: how many keys equal to the threshold are taken
        }
        mask |= digit_mask << low;
        top = low;
        __syncthreads();
    }
    const unsigned thr = sm.prefix + kmin;
    const int need_eq = sm.remaining;

    // ---- ordered compaction ----------------------------------------------------------
    int n_eq = 0, n_gt = 0;
    if (IN_REGS) {
#pragma unroll
        for (int e = 0; e < kTopkRegs; ++e)
            if (w_lo + e < w_hi) {
                n_eq += keys[e] == thr;
                n_gt += keys[e] > thr;
            }
    } else {
        for (int e = 0; w_lo + e < w_hi; ++e) {
            const unsigned key = key_at(e);
            n_eq += key == thr;
            n_gt += key > thr;
        }
    }
    int eq_rank, pos;   // threshold keys before this thread; output position of its first selected window
    if (IN_REGS) {
        // at most NT * 8 < 2^15 windows: both counts travel through one scan
        int total;
        const int both = topk_block_scan<NT>((n_eq << 16) | n_gt, sm.warp_sums, total);
        eq_rank = both >> 16;
        pos = (both & 0xffff) + (eq_rank < need_eq ? eq_rank : need_eq);
    } else {
        int eq_total, sel_total;
        eq_rank = topk_block_scan<NT>(n_eq, sm.warp_sums, eq_total);
        int n_eq_taken = need_eq - eq_rank;
        n_eq_taken = n_eq_taken < 0 ? 0 : (n_eq_taken > n_eq ? n_eq : n_eq_taken);
        pos = topk_block_scan<NT>(n_gt + n_eq_taken, sm.warp_sums, sel_total);
    }
    auto emit = [&](int e, unsigned key) {
        bool sel = key > thr;
        if (key == thr) {
            sel = eq_rank < need_eq;
            ++eq_rank;
        }
        if (sel) {
            out[pos++] = w_lo + e;
            if (w_lo + e == kw - 1) sm.last_selected = 1;
        }
    };
    if (IN_REGS) {
#pragma unroll
        for (int e = 0; e < kTopkRegs; ++e)
            if (w_lo + e < w_hi) emit(e, keys[e]);
    } else {
        for (int e = 0; w_lo + e < w_hi; ++e) emit(e, key_at(e));
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int n_r = n - alpha;
        const int last_size = n_r - (kw - 1) * omega;     // real size of the last window
        *kept_len_out = k * omega - (sm.last_selected ? omega - last_size : 0) + obs_rows;
    }
}

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
    const int per_thread = (kw + NT - 1) / NT;
    if (per_thread <= 4)
        select_topk_impl<NT, 4>(sm, sc, kw, k, out, kept_len_out, n, alpha, omega, obs_rows);
    else if (per_thread <= 8)
        select_topk_impl<NT, 8>(sm, sc, kw, k, out, kept_len_out, n, alpha, omega, obs_rows);
    else
        select_topk_impl<NT, 0>(sm, sc, kw, k, out, kept_len_out, n, alpha, omega, obs_rows);
}

}  // namespace wkv
