// Device-side pieces shared by the tensor-core score kernels: the per-element work of the two sweeps
// (Eq. 1's online statistics, Eq. 2's normalised sum), Eq. 4's pooling of one window, and the
// acquire / release accesses and bounded polls of the hand-over between thread blocks.
#pragma once

#include "tc_common.cuh"
#include "wkv_internal.cuh"

namespace wkv {
namespace {

using namespace tc;

__device__ __forceinline__ int ld_acquire_gpu(const int *p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_gpu_add(int *p, int v)
{
    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// one thread: polls until the word has reached `target`; false once the block has given up
// (`sleep_ns` > 0: the thread sleeps between looks, for waits that are expected to be long)
__device__ __forceinline__ bool poll_until_at_least(const int *word, int target, volatile int *abort_flag,
                                                    unsigned sleep_ns = 0)
{
    unsigned long long t0 = 0;
    for (uint32_t spin = 1; ld_acquire_gpu(word) < target; ++spin) {
        if (*abort_flag) return false;
        if (sleep_ns) __nanosleep(sleep_ns);
        if ((spin & 255u) == 0u) {
            const unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > 2 * kWaitLimitNs) {
                *abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ bool warp_wait_arrivals(const int *word, int target, volatile int *abort_flag, int lane)
{
    int ok = 1;
    if (lane == 0) ok = poll_until_at_least(word, target, abort_flag) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// ---------------------------------------------------------------------------------------------
// per-element work of the two sweeps
// ---------------------------------------------------------------------------------------------
// sweep 1: online-softmax update of one row with 32 more logits (raw dot products; c = log2(e)/sqrt(d))
__device__ __forceinline__ void stats_update(float (&v)[32], bool fast, int jb, int limit, float c, float &m,
                                             float &l)
{
    if (!fast) {
#pragma unroll
        for (int x = 0; x < 32; ++x)
            if (jb + x > limit) v[x] = -INFINITY;
    }
    float g0 = fmaxf(v[0], v[1]), g1 = fmaxf(v[2], v[3]);
#pragma unroll
    for (int x = 4; x < 32; x += 4) {
        g0 = fmaxf(g0, fmaxf(v[x], v[x + 1]));
        g1 = fmaxf(g1, fmaxf(v[x + 2], v[x + 3]));
    }
    const float m_new = fmaxf(m, fmaxf(g0, g1));
    if (m_new > -INFINITY) {
        const float mc = m_new * c;
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
        for (int x = 0; x < 32; x += 4) {
            a0 += fast_exp2(fmaf(v[x], c, -mc));
            a1 += fast_exp2(fmaf(v[x + 1], c, -mc));
            a2 += fast_exp2(fmaf(v[x + 2], c, -mc));
            a3 += fast_exp2(fmaf(v[x + 3], c, -mc));
        }
        const float add = (a0 + a1) + (a2 + a3);
        l = m_new == m ? l + add : l * fast_exp2((m - m_new) * c) + add;
        m = m_new;
    }
}
// sweep 2: adds exp2(x*c - lse2) of 32 (or 16) rows to the four partial sums of a key
template <int N>
__device__ __forceinline__ void score_accumulate(const float (&v)[N], const float *nl_base, float c, float &a0,
                                                 float &a1, float &a2, float &a3)
{
#pragma unroll
    for (int x = 0; x < N; x += 4) {
        const float4 nl = *reinterpret_cast<const float4 *>(nl_base + x);
        a0 += fast_exp2(fmaf(v[x], c, nl.x));
        a1 += fast_exp2(fmaf(v[x + 1], c, nl.y));
        a2 += fast_exp2(fmaf(v[x + 2], c, nl.z));
        a3 += fast_exp2(fmaf(v[x + 3], c, nl.w));
    }
}

// Eq. 4 for one window of compile-time length (a power of two) by one thread: a bitonic sorting
// network in registers (every compare-exchange of a stage is independent of the others, so the
// thread is not latency-bound), then the p largest are summed in descending order.  Positions
// beyond `size` (ragged last window) hold -inf and sort to the end.
template <int omega>
__device__ __forceinline__ float pool_window_sorted(const float *w, int size, int p)
{
    float v[omega];
#pragma unroll
    for (int x = 0; x < omega; ++x) v[x] = x < size ? w[x] : -INFINITY;
#pragma unroll
    for (int k = 2; k <= omega; k <<= 1)
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1)
#pragma unroll
            for (int i = 0; i < omega; ++i) {
                const int l = i ^ j;
                if (l > i) {
                    const float hi = fmaxf(v[i], v[l]), lo = fminf(v[i], v[l]);
                    const bool descending = (i & k) == 0;
                    v[i] = descending ? hi : lo;
                    v[l] = descending ? lo : hi;
                }
            }
    const int p_eff = p < size ? p : size;
    float acc = 0.f;
#pragma unroll
    for (int x = 0; x < omega; ++x) acc += x < p_eff ? v[x] : 0.f;
    return acc / (float)p_eff;
}

// Eq. 4 for one window of 64 or 128 tokens by one warp: lane l holds elements l, l + 32, ... in
// registers; a bitonic sorting network over (register, lane) orders them descending (partners 32 or
// more apart are registers of the same lane, closer ones are exchanged by shuffle), then the p largest
// are summed: per lane in ascending rank, across lanes by a fixed butterfly, so the result is the same
// from run to run.  Positions beyond `size` hold -inf.  Every lane returns the window score.
template <int omega>
__device__ __forceinline__ float pool_window_warp(const float *w, int size, int p, int lane)
{
    constexpr int NR = omega / 32;
    static_assert(omega == 64 || omega == 128, "window length");
    float v[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r) v[r] = r * 32 + lane < size ? w[r * 32 + lane] : -INFINITY;
#pragma unroll
    for (int k = 2; k <= omega; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            if (j >= 32) {
                const int jj = j >> 5;
#pragma unroll
                for (int r = 0; r < NR; ++r) {
                    if ((r & jj) == 0) {
                        const float hi = fmaxf(v[r], v[r | jj]), lo = fminf(v[r], v[r | jj]);
                        const bool descending = ((r * 32 + lane) & k) == 0;
                        v[r] = descending ? hi : lo;
                        v[r | jj] = descending ? lo : hi;
                    }
                }
            } else {
#pragma unroll
                for (int r = 0; r < NR; ++r) {
                    const float other = __shfl_xor_sync(0xffffffffu, v[r], j);
                    const bool lower = (lane & j) == 0;
                    const bool descending = ((r * 32 + lane) & k) == 0;
                    v[r] = (lower == descending) ? fmaxf(v[r], other) : fminf(v[r], other);
                }
            }
        }
    }
    const int p_eff = p < size ? p : size;
    float acc = 0.f;
#pragma unroll
    for (int r = 0; r < NR; ++r) acc += (r * 32 + lane < p_eff) ? v[r] : 0.f;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    return acc / (float)p_eff;
}

}  // namespace
}  // namespace wkv
