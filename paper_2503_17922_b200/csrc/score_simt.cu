// CUDA-core (FFMA) score kernels: Eq. 1-4 for fp32 inputs and for shapes the
// tensor-core kernels do not cover.  Two kernels per call:
//   stats : per row of the unit, partial (max, sum exp2) over a chunk of keys
//           (Eq. 1's normaliser, causal mask applied)
//   score : logits again, p = exp2(x - lse2), sum over the rows (Eq. 2), then the
//           Top-p window pooling of Eq. 3-4
// Summation orders are fixed, so results are bit-identical from run to run.
#include "wkv_internal.cuh"

#include <mutex>

#include <math.h>

namespace wkv {
namespace {

constexpr int kThreads = 256;
constexpr int kRT = 64;       // rows per logit tile
constexpr int kKT = 64;       // keys per logit tile
constexpr int kKPad = kKT + 4;

__device__ inline float to_float(float x) { return x; }
__device__ inline float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
struct Vec;  // 16-byte vector of T
template <>
struct Vec<float> {
    static constexpr int N = 4;
    float v[4];
};
template <>
struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    __nv_bfloat16 v[8];
};

template <typename T>
__device__ inline Vec<T> load_vec(const T *p)
{
    Vec<T> r;
    *reinterpret_cast<int4 *>(&r) = *reinterpret_cast<const int4 *>(p);
    return r;
}

// Q of the unit, transposed into shared memory: qs[c * r_pad + r]; rows >= R are zero.
template <typename T>
__device__ void load_q_transposed(const KShape &s, const T *q_unit, float *qs, int r_pad)
{
    constexpr int VN = Vec<T>::N;
    const int vec_per_row = s.d / VN;
    for (int idx = threadIdx.x; idx < r_pad * vec_per_row; idx += kThreads) {
        int r = idx / vec_per_row, cv = idx % vec_per_row;
        Vec<T> v;
        if (r < s.R) {
            int g = r / s.alpha, i = r % s.alpha;
            v = load_vec(q_unit + g * s.qsh + i * s.qst + cv * VN);
        } else {
#pragma unroll
            for (int e = 0; e < VN; ++e) v.v[e] = T(0.f);
        }
#pragma unroll
        for (int e = 0; e < VN; ++e) qs[(cv * VN + e) * r_pad + r] = to_float(v.v[e]);
    }
}

// kKT keys starting at j0, transposed: ks[c * kKPad + jj]; keys >= n_valid are zero.
template <typename T>
__device__ void load_k_transposed(const KShape &s, const T *k_unit, float *ks, int j0, int n_valid)
{
    constexpr int VN = Vec<T>::N;
    const int vec_per_row = s.d / VN;
    for (int idx = threadIdx.x; idx < kKT * vec_per_row; idx += kThreads) {
        int jj = idx / vec_per_row, cv = idx % vec_per_row;
        Vec<T> v;
        if (j0 + jj < n_valid) {
            v = load_vec(k_unit + (long long)(j0 + jj) * s.st + cv * VN);
        } else {
#pragma unroll
            for (int e = 0; e < VN; ++e) v.v[e] = T(0.f);
        }
#pragma unroll
        for (int e = 0; e < VN; ++e) ks[(cv * VN + e) * kKPad + jj] = to_float(v.v[e]);
    }
}

// 4x4 register tile of raw dot products for rows r0+ty*4.., keys tx*4..
__device__ inline void logits_4x4(const float *qs, const float *ks, int d, int r_pad, int r0, int ty,
                                  int tx, float acc[4][4])
{
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
    const float *qp = qs + r0 + ty * 4;
    const float *kp = ks + tx * 4;
#pragma unroll 4
    for (int c = 0; c < d; ++c) {
        float4 qv = *reinterpret_cast<const float4 *>(qp + c * r_pad);
        float4 kv = *reinterpret_cast<const float4 *>(kp + c * kKPad);
        float qa[4] = {qv.x, qv.y, qv.z, qv.w};
        float ka[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(qa[a], ka[b], acc[a][b]);
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
score_stats_simt(KShape s, const T *__restrict__ q, const T *__restrict__ k, float2 *__restrict__ stats,
                 int n_chunks, int r_pad)
{
    extern __shared__ __align__(16) float smem[];
    float *qs = smem;                    // [d][r_pad]
    float *ks = smem + s.d * r_pad;      // [d][kKPad]

    const int unit = blockIdx.y, chunk = blockIdx.x;
    const int b = unit / s.hkv, h = unit % s.hkv;
    const SeqInfo si = seq_info(s, b);
    const int n = si.n, n_r = n - s.alpha;
    float2 *out = stats + ((size_t)unit * n_chunks + chunk) * r_pad;
    const int j_begin = chunk * kStatChunk;
    if (n_r <= 0 || j_begin >= n) {
        for (int r = threadIdx.x; r < r_pad; r += kThreads) out[r] = make_float2(-INFINITY, 0.f);
        return;
    }
    const int j_end = min(n, j_begin + kStatChunk);
    const T *q_unit = q + b * s.qsb + (long long)h * s.G * s.qsh;
    const T *k_unit = k + (si.off * s.st + b * s.sb + h * s.sh);
    load_q_transposed(s, q_unit, qs, r_pad);

    const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
    for (int r0 = 0; r0 < r_pad; r0 += kRT) {
        float m[4], l[4];
        int pos[4];   // last key each row may attend to
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            m[a] = -INFINITY;
            l[a] = 0.f;
            int r = r0 + ty * 4 + a;
            pos[a] = r < s.R ? n_r + (r % s.alpha) : -1;
        }
        for (int j0 = j_begin; j0 < j_end; j0 += kKT) {
            __syncthreads();
            load_k_transposed(s, k_unit, ks, j0, n);
            __syncthreads();
            float acc[4][4];
            logits_4x4(qs, ks, s.d, r_pad, r0, ty, tx, acc);
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                float x[4], tmax = -INFINITY;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    int j = j0 + tx * 4 + c;
                    x[c] = j <= pos[a] ? acc[a][c] * s.scale_log2 : -INFINITY;
                    tmax = fmaxf(tmax, x[c]);
                }
#pragma unroll
                for (int o = 1; o < 16; o <<= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
                // no early exit: both half-warps must reach the shuffles below
                float m_new = fmaxf(m[a], tmax);
                float m_safe = m_new == -INFINITY ? 0.f : m_new;
                float sum = 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) sum += exp2f(x[c] - m_safe);
#pragma unroll
                for (int o = 1; o < 16; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                l[a] = l[a] * exp2f(m[a] - m_safe) + sum;
                m[a] = m_new;
            }
        }
        if (tx == 0) {
#pragma unroll
            for (int a = 0; a < 4; ++a) out[r0 + ty * 4 + a] = make_float2(m[a], l[a]);
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
score_pool_simt(KShape s, const T *__restrict__ q, const T *__restrict__ k,
                const float2 *__restrict__ stats, const float *__restrict__ lse_obs,
                float *__restrict__ window_scores, float *__restrict__ token_scores, int n_chunks, int r_pad,
                int chunk_keys)
{
    extern __shared__ __align__(16) float smem[];
    float *qs = smem;                          // [d][r_pad]
    float *ks = qs + s.d * r_pad;              // [d][kKPad]
    float *lse2 = ks + s.d * kKPad;            // [r_pad]
    float *part = lse2 + r_pad;                // [16][kKT]
    float *t_chunk = part + 16 * kKT;          // [chunk_keys rounded up to kKT]

    const int unit = blockIdx.y;
    const int b = unit / s.hkv, h = unit % s.hkv;
    const SeqInfo si = seq_info(s, b);
    const int n = si.n, n_r = n - s.alpha;
    const int j_begin = blockIdx.x * chunk_keys;
    if (n_r <= 0 || j_begin >= n_r) return;
    const int j_end = min(n_r, j_begin + chunk_keys);
    const T *q_unit = q + b * s.qsb + (long long)h * s.G * s.qsh;
    const T *k_unit = k + (si.off * s.st + b * s.sb + h * s.sh);
    load_q_transposed(s, q_unit, qs, r_pad);

    // combine the partial statistics of every chunk: lse2 = log2 of the row normaliser
    // (or, when the caller supplies the natural log of the normalisers, that value in base 2)
    for (int r = threadIdx.x; r < r_pad; r += kThreads) {
        if (lse_obs) {
            const int g = r / s.alpha, i = r - g * s.alpha;
            lse2[r] = r < s.R ? lse_obs[((size_t)b * s.hq + (size_t)h * s.G + g) * s.alpha + i] * 1.4426950408889634f
                              : INFINITY;
            continue;
        }
        const float2 *st = stats + (size_t)unit * n_chunks * r_pad + r;
        float M = -INFINITY;
        for (int c = 0; c < n_chunks; ++c) M = fmaxf(M, st[(size_t)c * r_pad].x);
        float L = 0.f;
        for (int c = 0; c < n_chunks; ++c) {
            float2 v = st[(size_t)c * r_pad];
            if (v.y > 0.f) L += v.y * exp2f(v.x - M);
        }
        lse2[r] = (r < s.R && L > 0.f) ? M + log2f(L) : INFINITY;
    }

    const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
    for (int j0 = j_begin; j0 < j_end; j0 += kKT) {
        __syncthreads();
        load_k_transposed(s, k_unit, ks, j0, n_r);
        __syncthreads();
        float t_acc = 0.f;   // threads 0..kKT-1: token score of key j0 + tid
        for (int r0 = 0; r0 < r_pad; r0 += kRT) {
            float acc[4][4];
            logits_4x4(qs, ks, s.d, r_pad, r0, ty, tx, acc);
            float col[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                float ls = lse2[r0 + ty * 4 + a];
#pragma unroll
                for (int c = 0; c < 4; ++c) col[c] += exp2f(fmaf(acc[a][c], s.scale_log2, -ls));
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) part[ty * kKT + tx * 4 + c] = col[c];
            __syncthreads();
            if (threadIdx.x < kKT) {
#pragma unroll
                for (int y = 0; y < 16; ++y) t_acc += part[y * kKT + threadIdx.x];
            }
            __syncthreads();
        }
        if (threadIdx.x < kKT) {
            int j = j0 + threadIdx.x;
            t_chunk[j - j_begin] = t_acc;
            if (token_scores && j < n_r) token_scores[(size_t)unit * s.nr_max + j] = t_acc;
        }
    }
    __syncthreads();
    // Eq. 3-4: windows of this chunk (chunk_keys is a multiple of omega)
    const int w_begin = j_begin / s.omega;
    const int n_win = (j_end - j_begin + s.omega - 1) / s.omega;
    for (int lw = threadIdx.x; lw < n_win; lw += kThreads) {
        int lo = lw * s.omega;
        int size = min(s.omega, (j_end - j_begin) - lo);
        window_scores[(size_t)unit * s.kw_max + w_begin + lw] = pool_top_p(t_chunk + lo, size, s.p);
    }
}

}  // namespace

// The opt-in to more than 48 KB of dynamic shared memory is a property of (kernel, device): it is
// raised once per device and kernel to the largest size asked for so far, not on every launch.
static cudaError_t allow_dynamic_smem(const void *fn, int dev, int slot, size_t bytes)
{
    static std::mutex mu;
    static size_t allowed[kMaxDevices][4] = {};
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (bytes <= allowed[dev][slot]) return cudaSuccess;
    const cudaError_t err = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (err == cudaSuccess) allowed[dev][slot] = bytes;
    return err;
}

static int simt_chunk_keys(const KShape &ks)
{
    int per = 512 / ks.omega;
    if (per < 1) per = 1;
    return per * ks.omega;
}

cudaError_t launch_score_simt(const KShape &ks, int dtype, const void *q, const void *k,
                              float *window_scores, float *token_scores,
                              void *workspace, const Workspace &ws, cudaStream_t stream, const float *lse_obs)
{
    const int units = ks.batch * ks.hkv;
    const int r_pad = ws.r_pad;
    float2 *stats = reinterpret_cast<float2 *>(static_cast<char *>(workspace) + ws.stats_off);
    const int chunk_keys = simt_chunk_keys(ks);
    const int n_r_max = ks.max_seqlen - ks.alpha;
    if (n_r_max <= 0) return cudaSuccess;
    const int n_score_chunks = (n_r_max + chunk_keys - 1) / chunk_keys;
    const size_t smem1 = sizeof(float) * ((size_t)ks.d * r_pad + (size_t)ks.d * kKPad);
    const size_t smem2 = smem1 + sizeof(float) * ((size_t)r_pad + 16 * kKT +
                                                  (size_t)((chunk_keys + kKT - 1) / kKT) * kKT);
    dim3 g1(ws.n_stat_chunks, units), g2(n_score_chunks, units);
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
#define WKV_LAUNCH_SIMT(T, SLOT)                                                                    \
    do {                                                                                            \
        err = allow_dynamic_smem(reinterpret_cast<const void *>(score_stats_simt<T>), dev, SLOT, smem1);     \
        if (err != cudaSuccess) return err;                                                         \
        err = allow_dynamic_smem(reinterpret_cast<const void *>(score_pool_simt<T>), dev, SLOT + 1, smem2);  \
        if (err != cudaSuccess) return err;                                                         \
        if (!lse_obs)                                                                               \
            score_stats_simt<T><<<g1, kThreads, smem1, stream>>>(ks, (const T *)q, (const T *)k, stats, \
                                                                 ws.n_stat_chunks, r_pad);          \
        score_pool_simt<T><<<g2, kThreads, smem2, stream>>>(ks, (const T *)q, (const T *)k, stats,  \
                                                            lse_obs, window_scores, token_scores,   \
                                                            ws.n_stat_chunks, r_pad, chunk_keys);   \
    } while (0)
    if (dtype == WKV_F32)
        WKV_LAUNCH_SIMT(float, 0);
    else
        WKV_LAUNCH_SIMT(__nv_bfloat16, 2);
#undef WKV_LAUNCH_SIMT
    count_launches(lse_obs ? 1 : 2);
    return cudaGetLastError();
}

// shared-memory need of the CUDA-core kernels, for the host-side support check
size_t score_simt_smem_bytes(const KShape &ks, int r_pad)
{
    const int chunk_keys = simt_chunk_keys(ks);
    return sizeof(float) * ((size_t)ks.d * r_pad + (size_t)ks.d * kKPad + (size_t)r_pad + 16 * kKT +
                            (size_t)((chunk_keys + kKT - 1) / kKT) * kKT);
}

}  // namespace wkv
