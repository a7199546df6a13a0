// Budgeted window selection (sentence after Eq. 4) for one unit by one thread block: the k-th
// largest window score is found with a radix select (9 bits per pass, only over the bits in which
// the unit's keys differ, finished by direct ranking once few candidates are left) over an
// order-preserving integer image of the fp32 scores, then the selected window indices are emitted
// in ascending order with one block-wide prefix sum.  Equal scores at the threshold go to the
// lower window index.  Integer arithmetic only after the key mapping, so the result is exact and
// deterministic.  Used by the stand-alone selection kernel and by the fused score kernel.
//
// The whole selection is a chain of short dependent steps, so it is written for latency: block-wide
// reductions go through one word per warp and one warp-reduce instruction per reader (one barrier
// each), the histogram of a pass is small enough for a single warp to search, and no step waits on
// the return value of a shared-memory atomic except one per warp in the direct finish.
#pragma once

#include "wkv_internal.cuh"

namespace wkv {

constexpr int kTopkDigit = 9;                 // bits resolved per pass
constexpr int kTopkBins = 1 << kTopkDigit;    // 16 bins per lane of the warp that searches the histogram
constexpr int kTopkDirect = 64;               // with at most this many candidates left, rank them directly

struct TopkSmem {
    __align__(16) int hist[kTopkBins];
    __align__(16) unsigned cand[kTopkDirect];
    int warp_sums[2][32];       // two slots: consecutive block scans need no barrier between them
    unsigned warp_min[32], warp_max[32];
    unsigned prefix;
    int remaining;
    int last_selected;
    int cand_total, n_cand;     // keys in the chosen bin; candidates collected for the direct finish
};

// The NT threads that take part are threads TID0 .. TID0 + NT - 1 of the block.  BAR = 0: they are the
// whole block and synchronise with the block barrier; BAR > 0: they are a subset of the block's warps
// and synchronise on named barrier BAR (the rest of the block runs on independently).
template <int TID0>
__device__ __forceinline__ int topk_tid()
{
    return (int)threadIdx.x - TID0;
}
template <int NT, int BAR>
__device__ __forceinline__ void topk_sync()
{
    if (BAR == 0) __syncthreads();
    else asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(NT) : "memory");
}

// larger float <=> larger key; -0 and +0 map to the same key
__device__ __forceinline__ unsigned topk_order_key(float f)
{
    unsigned u = __float_as_uint(f);
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ int topk_warp_scan(int v, int lane)   // inclusive
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Exclusive prefix sum of `v` over the NT threads of the block; also returns the total.  One word
// written per warp, one barrier, then every warp adds up the totals of the warps before it with a
// warp-reduce instruction.  `warp_sums` (32 words) must not be in use by a scan that some thread
// of the block may not have left yet: alternate between two slots.
template <int NT, int BAR, int TID0>
__device__ __forceinline__ int topk_block_scan(int v, int *warp_sums, int &total)
{
    constexpr int kWarps = NT / 32;
    const int lane = topk_tid<TID0>() & 31, warp = topk_tid<TID0>() >> 5;
    const int incl = topk_warp_scan(v, lane);
    if (lane == 31) warp_sums[warp] = incl;
    topk_sync<NT, BAR>();
    const int wt = lane < kWarps ? warp_sums[lane] : 0;
    total = __reduce_add_sync(0xffffffffu, wt);
    return __reduce_add_sync(0xffffffffu, lane < warp ? wt : 0) + incl - v;
}

// All NT threads of the block call this.  `sc` are the unit's kw window scores (read through L2,
// so scores written by other blocks of the same grid are seen once the caller has synchronised
// with them), `out` receives k ascending indices followed by -1 up to k_max.
// Thread t owns the windows [t*E, (t+1)*E), E = ceil(kw / NT).  With E <= REGS (4 or 8) the keys
// are read once and stay in registers through the radix passes and the compaction (one trip to L2
// instead of several); REGS = 0: longer lists are re-read.
template <int NT, int REGS, int BAR, int TID0>
__device__ __forceinline__ void select_topk_impl(TopkSmem &sm, const float *sc, int kw, int k, int *out,
                                                 int *kept_len_out, int n, int alpha, int omega, int obs_rows)
{
    constexpr int kWarps = NT / 32;
    static_assert(NT % 32 == 0 && NT >= kTopkDirect, "block size");
    const int lane = topk_tid<TID0>() & 31, warp = topk_tid<TID0>() >> 5;
    const int E = (kw + NT - 1) / NT;
    const int w_lo = min(kw, (int)topk_tid<TID0>() * E), w_hi = min(kw, w_lo + E);
    constexpr bool IN_REGS = REGS > 0;
    constexpr int kTopkRegs = IN_REGS ? REGS : 1;
    unsigned keys[kTopkRegs];
    if (IN_REGS) {
#pragma unroll
        for (int e = 0; e < kTopkRegs; ++e) keys[e] = w_lo + e < w_hi ? topk_order_key(__ldcg(sc + w_lo + e)) : 0u;
    }
    auto key_at = [&](int e) -> unsigned { return IN_REGS ? keys[e] : topk_order_key(__ldcg(sc + w_lo + e)); };
    // runs f(e, key) over the thread's own keys
    auto for_own = [&](auto f) {
        if (IN_REGS) {
#pragma unroll
            for (int e = 0; e < kTopkRegs; ++e)
                if (w_lo + e < w_hi) f(e, keys[e]);
        } else {
            for (int e = 0; w_lo + e < w_hi; ++e) f(e, key_at(e));
        }
    };

    // ---- radix select: key of the k-th largest score --------------------------------
    // Keys are taken relative to the smallest one, and only the bits in which the largest differs
    // from it are resolved, 9 at a time from the top (window scores share sign and most of the
    // exponent: typically one pass), until at most kTopkDirect candidates share the prefix; those
    // are ranked against each other directly.
    if (topk_tid<TID0>() == 0) {
        sm.prefix = 0u;
        sm.remaining = k;
        sm.last_selected = 0;
        sm.cand_total = kw;
        sm.n_cand = 0;
    }
    for (int x = topk_tid<TID0>(); x < kTopkBins; x += NT) sm.hist[x] = 0;
    unsigned kmin, kmax;
    {
        unsigned lo = 0xffffffffu, hi = 0u;
        for_own([&](int, unsigned key) {
            lo = min(lo, key);
            hi = max(hi, key);
        });
        lo = __reduce_min_sync(0xffffffffu, lo);
        hi = __reduce_max_sync(0xffffffffu, hi);
        if (lane == 0) {
            sm.warp_min[warp] = lo;
            sm.warp_max[warp] = hi;
        }
        topk_sync<NT, BAR>();
        kmin = __reduce_min_sync(0xffffffffu, lane < kWarps ? sm.warp_min[lane] : 0xffffffffu);
        kmax = __reduce_max_sync(0xffffffffu, lane < kWarps ? sm.warp_max[lane] : 0u);
    }
    const int bits = 32 - __clz(kmax - kmin);        // 0 when all keys are equal
    unsigned mask = 0u;
    int top = bits;                                   // bits [top, 32) of (key - kmin) are resolved
#pragma unroll 1
    while (top > 0) {
        const unsigned prefix = sm.prefix;
        const int remaining = sm.remaining;
        if (sm.cand_total <= kTopkDirect) {
            // direct finish: the candidates are collected (one atomic per warp that holds any) and
            // each is ranked against the others
            int cnt = 0;
            for_own([&](int, unsigned key) { cnt += ((key - kmin) & mask) == prefix; });
            const int incl = topk_warp_scan(cnt, lane);
            int base = 0;
            if (lane == 31 && incl > 0) base = atomicAdd(&sm.n_cand, incl);
            int slot = __shfl_sync(0xffffffffu, base, 31) + incl - cnt;
            for_own([&](int, unsigned key) {
                const unsigned rk = key - kmin;
                if ((rk & mask) == prefix) sm.cand[slot++] = rk;
            });
            topk_sync<NT, BAR>();
            const int n_cand = sm.n_cand;
            if ((int)topk_tid<TID0>() < n_cand) {
                const unsigned my = sm.cand[topk_tid<TID0>()];
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
            topk_sync<NT, BAR>();
            break;
        }
        const int low = top > kTopkDigit ? top - kTopkDigit : 0;
        const unsigned digit_mask = (1u << (top - low)) - 1u;
        for_own([&](int, unsigned key) {
            const unsigned rk = key - kmin;
            if ((rk & mask) == prefix) atomicAdd(&sm.hist[(rk >> low) & digit_mask], 1);
        });
        topk_sync<NT, BAR>();
        if (warp == 0) {
            // the bin (from the top) in which the count reaches `remaining`: lane l holds bins 16 l .. 16 l + 15
            int c[16], mine = 0;
            int4 *hv = reinterpret_cast<int4 *>(sm.hist + lane * 16);
#pragma unroll
            for (int i = 0; i < 16; i += 4) {
                const int4 x = hv[i / 4];
                hv[i / 4] = make_int4(0, 0, 0, 0);   // ready for the next pass
                c[i] = x.x;
                c[i + 1] = x.y;
                c[i + 2] = x.z;
                c[i + 3] = x.w;
                mine += (x.x + x.y) + (x.z + x.w);
            }
            int upto = mine;                          // keys in this lane's bins and in higher lanes' bins
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_down_sync(0xffffffffu, upto, o);
                if (lane + o < 32) upto += t;
            }
            const int above = upto - mine;
            if (above < remaining && remaining <= upto) {
                int rem = remaining - above, bin = lane * 16;
#pragma unroll
                for (int i = 15; i >= 0; --i) {
                    if (c[i] >= rem) {
                        bin = lane * 16 + i;
                        sm.cand_total = c[i];
                        break;
                    }
                    rem -= c[i];
                }
                sm.prefix = prefix | ((unsigned)bin << low);
                sm.remaining = rem;   // after the last pass: how many keys equal to the threshold are taken
            }
        }
        mask |= digit_mask << low;
        top = low;
        topk_sync<NT, BAR>();
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
        const int both = topk_block_scan<NT, BAR, TID0>((n_eq << 16) | n_gt, sm.warp_sums[0], total);
        eq_rank = both >> 16;
        pos = (both & 0xffff) + (eq_rank < need_eq ? eq_rank : need_eq);
    } else {
        int eq_total, sel_total;
        eq_rank = topk_block_scan<NT, BAR, TID0>(n_eq, sm.warp_sums[0], eq_total);
        int n_eq_taken = need_eq - eq_rank;
        n_eq_taken = n_eq_taken < 0 ? 0 : (n_eq_taken > n_eq ? n_eq : n_eq_taken);
        pos = topk_block_scan<NT, BAR, TID0>(n_gt + n_eq_taken, sm.warp_sums[1], sel_total);
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
    topk_sync<NT, BAR>();
    if (topk_tid<TID0>() == 0) {
        const int n_r = n - alpha;
        const int last_size = n_r - (kw - 1) * omega;     // real size of the last window
        *kept_len_out = k * omega - (sm.last_selected ? omega - last_size : 0) + obs_rows;
    }
}

template <int NT, int BAR = 0, int TID0 = 0>
__device__ void select_topk_block(TopkSmem &sm, const float *sc, int kw, int k, int k_max, int *out,
                                  int *kept_len_out, int n, int alpha, int omega)
{
    static_assert(NT % 32 == 0 && NT <= 1024, "block size");
    for (int x = (k > 0 ? k : 0) + topk_tid<TID0>(); x < k_max; x += NT) out[x] = -1;
    const int obs_rows = n < alpha ? n : alpha;
    if (k <= 0) {
        if (topk_tid<TID0>() == 0) *kept_len_out = obs_rows;
        return;
    }
    const int per_thread = (kw + NT - 1) / NT;
    if (per_thread <= 4)
        select_topk_impl<NT, 4, BAR, TID0>(sm, sc, kw, k, out, kept_len_out, n, alpha, omega, obs_rows);
    else if (per_thread <= 8)
        select_topk_impl<NT, 8, BAR, TID0>(sm, sc, kw, k, out, kept_len_out, n, alpha, omega, obs_rows);
    else
        select_topk_impl<NT, 0, BAR, TID0>(sm, sc, kw, k, out, kept_len_out, n, alpha, omega, obs_rows);
}

}  // namespace wkv
