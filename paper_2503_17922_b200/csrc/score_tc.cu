// Tensor-core score kernels (tcgen05 + tensor memory + TMA) for bf16 inputs: Eq. 1-4 of the leader.
//
// The token score of Eq. 2, t_j = sum_i exp(s_ij) / Z_i, needs every row's softmax normaliser
// Z_i (a reduction over all keys) before any column sum can be finished, so the keys are swept
// twice:
//   score_stats_tc  sweep 1.  D[rows, keys] = Q K^T per 128-key tile with the observation rows on
//                   the tensor-memory lanes: one thread owns one row and keeps its running
//                   (max, sum exp2) without any cross-thread traffic (Eq. 1's normaliser, causal
//                   mask on the tiles that touch the observation window).  K comes from HBM.
//   score_pool_tc   sweep 2.  D[keys, rows] = K Q^T with the keys on the lanes: one thread owns one
//                   key and sums exp2(x_ij - lse2_i) over the rows (Eq. 2), the block then pools its
//                   windows (Eq. 3-4).  K comes from L2 when the leader's keys fit there.
// Both kernels are warp-specialised: warp 0 issues the TMA tile loads (4-stage ring), warp 1
// issues the MMAs into a double-buffered accumulator in tensor memory, warps 4-7 and 8-11 are two
// compute groups that take alternate tiles.  The contraction is the only tensor-core work; the
// exponentials, sums and the pooling are fp32 on the CUDA cores, in a fixed order.
#include "tc_common.cuh"
#include "wkv_internal.cuh"

#include <cuda.h>

#include <algorithm>
#include <mutex>

namespace wkv {
namespace {

using namespace tc;

constexpr int kThreads = 384;
constexpr int kStages = 4;
constexpr int kTile = kTcTileKeys;                       // keys per tile
constexpr int kRegion = kTile * 128;                     // bytes of one 64-column block of a key tile
constexpr int kChunkCap = kTcMaxChunkTiles * kTile + kTcMaxWindow;   // token scores a block may hold

struct TcArgs {
    KShape s;
    float2 *stats;          // [units][n_stat_chunks][r_pad]
    float *window_scores;
    float *token_scores;
    int *status;
    int n_stat_chunks, r_pad;
    int chunks_per_unit;
    int kblocks;            // head_dim / 64
    int slot_tok, slot_h, slot_b;   // which tensor-map coordinate (1..3) carries token / head / batch
    int r16;                // observation rows rounded up to a multiple of 16
    int tmem_cols;          // tensor-memory columns of the scoring kernel
};

__device__ __forceinline__ uint8_t *align_1024(uint8_t *p)
{
    return reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(p) + 1023u) & ~uintptr_t(1023u));
}

struct Barriers {
    uint64_t full[kStages];    // TMA -> MMA: the stage holds a key tile
    uint64_t empty[kStages];   // MMA -> TMA: the MMAs that read the stage have completed
    uint64_t tfull[2];         // MMA -> compute group: the accumulator buffer is complete
    uint64_t tempty[2];        // compute group -> MMA: the accumulator buffer has been read
};

__device__ __forceinline__ void init_barriers(Barriers &bar)
{
    for (int i = 0; i < kStages; ++i) {
        mbar_init(&bar.full[i], 1);
        mbar_init(&bar.empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
        mbar_init(&bar.tfull[i], 1);
        mbar_init(&bar.tempty[i], 128);
    }
    fence_barrier_init();
}

// Producer loop: key tiles t = 0 .. n_tiles-1 of the block into the stage ring, then waits until the
// last MMAs have released their stages (so nothing is in flight when the block ends).
__device__ __forceinline__ void produce_tiles(const CUtensorMap *tmap, const TcArgs &a, Barriers &bar,
                                              uint8_t *k_stage0, int n_tiles, int tok0, int h, int bcoord,
                                              volatile int *abort_flag)
{
    const int stage_bytes = a.kblocks * kRegion;
    tma_prefetch_desc(tmap);
    int issued = 0;
    for (int t = 0; t < n_tiles; ++t) {
        const int st = t % kStages;
        if (t >= kStages && !mbar_wait(&bar.empty[st], ((t / kStages) - 1) & 1, abort_flag)) break;
        mbar_arrive_expect_tx(&bar.full[st], (uint32_t)stage_bytes);
        const int tok = tok0 + t * kTile;
        const int c1 = a.slot_tok == 1 ? tok : (a.slot_h == 1 ? h : bcoord);
        const int c2 = a.slot_tok == 2 ? tok : (a.slot_h == 2 ? h : bcoord);
        const int c3 = a.slot_tok == 3 ? tok : (a.slot_h == 3 ? h : bcoord);
        for (int kb = 0; kb < a.kblocks; ++kb)
            tma_load_4d(k_stage0 + st * stage_bytes + kb * kRegion, tmap, &bar.full[st], kb * 64, c1, c2, c3);
        ++issued;
    }
    for (int t = issued > kStages ? issued - kStages : 0; t < issued; ++t) {
        const int st = t % kStages;
        if (!mbar_wait(&bar.empty[st], (t / kStages) & 1, abort_flag)) {
            // giving up: the loads already issued must still land before the block may end
            volatile int never = 0;
            mbar_wait(&bar.full[st], (t / kStages) & 1, &never);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// sweep 1: per-row partial (max, sum exp2) over the block's keys
// ---------------------------------------------------------------------------------------------
template <int MB>   // 128-row blocks of observation rows: 1 (R <= 128) or 2 (R <= 256)
__global__ void __launch_bounds__(kThreads, 1)
score_stats_tc(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ TcArgs a,
               const __nv_bfloat16 *__restrict__ q)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) Barriers bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ float2 part[2][MB][128];

    const KShape &s = a.s;
    const int unit = blockIdx.y, chunk = blockIdx.x;
    const int b = unit / s.hkv, h = unit % s.hkv;
    const SeqInfo si = seq_info(s, b);
    const int n = si.n, n_r = n - s.alpha;
    float2 *out = a.stats + ((size_t)unit * a.n_stat_chunks + chunk) * a.r_pad;
    const int len = tc_chunk_len(n, a.chunks_per_unit, 1);
    const int j_begin = chunk * len;
    if (n_r <= 0 || j_begin >= n) {
        for (int r = threadIdx.x; r < a.r_pad; r += kThreads) out[r] = make_float2(-INFINITY, 0.f);
        return;
    }
    const int j_end = min(n, j_begin + len);
    const int n_tiles = (j_end - j_begin + kTile - 1) / kTile;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    uint8_t *q_img = align_1024(smem_raw);
    constexpr int q_rows = MB * 128;
    constexpr int q_region = q_rows * 128;
    uint8_t *k_stage0 = q_img + a.kblocks * q_region;
    const int stage_bytes = a.kblocks * kRegion;
    constexpr uint32_t tmem_cols = MB * 256;    // two accumulator buffers of MB x 128 columns

    if (threadIdx.x == 0) {
        init_barriers(bar);
        abort_s = 0;
    }
    if (warp == 1) tmem_alloc(&tmem_base_s, tmem_cols);

    // Q image: row r of the image is observation row (r mod Rp); with Rp < 128 the rows repeat so
    // that all 128 lanes work, each copy taking its own slice of a tile's columns
    const int Rp = MB == 2 ? 256 : (s.R <= 32 ? 32 : (s.R <= 64 ? 64 : 128));
    const __nv_bfloat16 *q_unit = q + b * s.qsb + (long long)h * s.G * s.qsh;
    const int vec_per_row = s.d / 8;
    for (int idx = threadIdx.x; idx < q_rows * vec_per_row; idx += kThreads) {
        const int r = idx / vec_per_row, cc = idx % vec_per_row;
        const int rq = r % Rp;
        int4 v = make_int4(0, 0, 0, 0);
        if (rq < s.R) {
            const int g = rq / s.alpha, i = rq % s.alpha;
            v = *reinterpret_cast<const int4 *>(q_unit + g * s.qsh + i * s.qst + cc * 8);
        }
        *reinterpret_cast<int4 *>(q_img + (cc >> 3) * q_region + swz128_offset(r, cc & 7)) = v;
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_s;

    if (warp == 0) {
        if (lane == 0)
            produce_tiles(&tmap, a, bar, k_stage0, n_tiles, (int)si.off + j_begin, h, s.cu ? 0 : b, &abort_s);
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, kTile);
            const uint32_t q_addr = smem_u32(q_img);
            const int ksteps = s.d / 16;
            for (int t = 0; t < n_tiles; ++t) {
                const int st = t % kStages, buf = t & 1;
                if (!mbar_wait(&bar.full[st], (t / kStages) & 1, &abort_s)) break;
                if (t >= 2 && !mbar_wait(&bar.tempty[buf], ((t >> 1) - 1) & 1, &abort_s)) break;
                tc_fence_after_sync();
                const uint32_t k_addr = smem_u32(k_stage0 + st * stage_bytes);
#pragma unroll
                for (int mb = 0; mb < MB; ++mb) {
                    const uint32_t d_tmem = tmem_base + buf * (MB * 128) + mb * 128;
                    for (int ks = 0; ks < ksteps; ++ks) {
                        const uint32_t kb = ks >> 2, sub = (ks & 3) * 32;
                        umma_bf16(d_tmem, umma_desc_sw128(q_addr + kb * q_region + mb * kRegion + sub),
                                  umma_desc_sw128(k_addr + kb * kRegion + sub), idesc, ks > 0);
                    }
                }
                umma_commit(&bar.empty[st]);
                umma_commit(&bar.tfull[buf]);
            }
        }
    } else if (warp >= 4) {
        const int grp = (warp - 4) >> 2, quarter = warp & 3;
        const int L = quarter * 32 + lane;
        const int ncols = MB == 2 ? kTile : Rp;             // columns of a tile this thread reduces
        const int col0 = MB == 2 ? 0 : (L / Rp) * Rp;       // warp-uniform: Rp is a multiple of 32
        const float c = s.scale_log2;
        float m[MB], l[MB];
        int limit[MB];                                      // last key the row may attend to
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) {
            m[mb] = -INFINITY;
            l[mb] = 0.f;
            const int row = MB == 2 ? mb * 128 + L : L % Rp;
            limit[mb] = row < s.R ? min(n_r + row % s.alpha, j_end - 1) : -1;
        }
        for (int t = grp; t < n_tiles; t += 2) {
            bool ok = mbar_wait(&bar.tfull[grp], (t >> 1) & 1, &abort_s);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const int j0 = j_begin + t * kTile;
            const bool fast = (j0 + kTile - 1 <= n_r) && (j0 + kTile - 1 < j_end);   // no masking needed
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + grp * (MB * 128) + mb * 128 + col0;
                for (int cg = 0; cg < ncols; cg += 32) {
                    float v[32];
                    tmem_ld32(taddr + cg, v);
                    if (!fast) {
                        const int jb = j0 + col0 + cg;
#pragma unroll
                        for (int x = 0; x < 32; ++x)
                            if (jb + x > limit[mb]) v[x] = -INFINITY;
                    }
                    float g0 = fmaxf(v[0], v[1]), g1 = fmaxf(v[2], v[3]);
#pragma unroll
                    for (int x = 4; x < 32; x += 4) {
                        g0 = fmaxf(g0, fmaxf(v[x], v[x + 1]));
                        g1 = fmaxf(g1, fmaxf(v[x + 2], v[x + 3]));
                    }
                    const float m_new = fmaxf(m[mb], fmaxf(g0, g1));
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
                        l[mb] = l[mb] * fast_exp2((m[mb] - m_new) * c) + ((a0 + a1) + (a2 + a3));
                        m[mb] = m_new;
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(&bar.tempty[grp]);
        }
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) part[grp][mb][L] = make_float2(m[mb], l[mb]);
    }

    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (!abort_s) {
        // combine the two compute groups and the column slices of each row, in a fixed order
        const float c = s.scale_log2;
        const int copies = MB == 2 ? 1 : 128 / Rp;
        for (int r = threadIdx.x; r < a.r_pad; r += kThreads) {
            float2 res = make_float2(-INFINITY, 0.f);
            if (r < s.R) {
                const int mb = MB == 2 ? r >> 7 : 0, base = MB == 2 ? (r & 127) : r;
                float M = -INFINITY;
                for (int g = 0; g < 2; ++g)
                    for (int cp = 0; cp < copies; ++cp) M = fmaxf(M, part[g][mb][base + cp * Rp].x);
                float sum = 0.f;
                for (int g = 0; g < 2; ++g)
                    for (int cp = 0; cp < copies; ++cp) {
                        const float2 p = part[g][mb][base + cp * Rp];
                        if (p.y > 0.f) sum += p.y * exp2f((p.x - M) * c);
                    }
                res = make_float2(M * c, sum);
            }
            out[r] = res;
        }
    } else if (threadIdx.x == 0) {
        atomicOr(a.status, kStatusWaitExpired);
    }
    if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);
}

// ---------------------------------------------------------------------------------------------
// sweep 2: token scores (Eq. 2) and window pooling (Eq. 3-4)
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1)
score_pool_tc(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ TcArgs a,
              const __nv_bfloat16 *__restrict__ q)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) Barriers bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ __align__(16) float neg_lse2[256];     // -log2 of the row normaliser; -inf for padding rows
    __shared__ float t_chunk[kChunkCap];

    const KShape &s = a.s;
    const int unit = blockIdx.y, chunk = blockIdx.x;
    const int b = unit / s.hkv, h = unit % s.hkv;
    const SeqInfo si = seq_info(s, b);
    const int n = si.n, n_r = n - s.alpha;
    if (n_r <= 0) return;
    const int len = tc_chunk_len(n_r, a.chunks_per_unit, s.omega);
    const int j_begin = chunk * len;
    if (j_begin >= n_r) return;
    const int j_end = min(n_r, j_begin + len);
    const int n_tiles = (j_end - j_begin + kTile - 1) / kTile;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    uint8_t *q_img = align_1024(smem_raw);
    const int q_region = a.r16 * 128;
    uint8_t *k_stage0 = align_1024(q_img + a.kblocks * q_region);
    const int stage_bytes = a.kblocks * kRegion;
    const int buf_cols = a.tmem_cols >> 1;

    if (threadIdx.x == 0) {
        init_barriers(bar);
        abort_s = 0;
    }
    if (warp == 1) tmem_alloc(&tmem_base_s, (uint32_t)a.tmem_cols);

    const __nv_bfloat16 *q_unit = q + b * s.qsb + (long long)h * s.G * s.qsh;
    const int vec_per_row = s.d / 8;
    for (int idx = threadIdx.x; idx < a.r16 * vec_per_row; idx += kThreads) {
        const int r = idx / vec_per_row, cc = idx % vec_per_row;
        int4 v = make_int4(0, 0, 0, 0);
        if (r < s.R) {
            const int g = r / s.alpha, i = r % s.alpha;
            v = *reinterpret_cast<const int4 *>(q_unit + g * s.qsh + i * s.qst + cc * 8);
        }
        *reinterpret_cast<int4 *>(q_img + (cc >> 3) * q_region + swz128_offset(r, cc & 7)) = v;
    }
    // Eq. 1's normaliser of every row from the partial statistics of sweep 1
    {
        const int len1 = tc_chunk_len(n, a.chunks_per_unit, 1);
        const int used = (n + len1 - 1) / len1;
        for (int r = threadIdx.x; r < 256; r += kThreads) {
            float v = -INFINITY;
            if (r < s.R) {
                const float2 *st = a.stats + (size_t)unit * a.n_stat_chunks * a.r_pad + r;
                float M = -INFINITY;
                for (int cidx = 0; cidx < used; ++cidx) M = fmaxf(M, st[(size_t)cidx * a.r_pad].x);
                float sum = 0.f;
                for (int cidx = 0; cidx < used; ++cidx) {
                    const float2 p = st[(size_t)cidx * a.r_pad];
                    if (p.y > 0.f) sum += p.y * exp2f(p.x - M);
                }
                if (sum > 0.f) v = -(M + log2f(sum));
            }
            neg_lse2[r] = v;
        }
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_s;

    if (warp == 0) {
        if (lane == 0)
            produce_tiles(&tmap, a, bar, k_stage0, n_tiles, (int)si.off + j_begin, h, s.cu ? 0 : b, &abort_s);
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(128, a.r16);
            const uint32_t q_addr = smem_u32(q_img);
            const int ksteps = s.d / 16;
            for (int t = 0; t < n_tiles; ++t) {
                const int st = t % kStages, buf = t & 1;
                if (!mbar_wait(&bar.full[st], (t / kStages) & 1, &abort_s)) break;
                if (t >= 2 && !mbar_wait(&bar.tempty[buf], ((t >> 1) - 1) & 1, &abort_s)) break;
                tc_fence_after_sync();
                const uint32_t k_addr = smem_u32(k_stage0 + st * stage_bytes);
                const uint32_t d_tmem = tmem_base + buf * buf_cols;
                for (int ks = 0; ks < ksteps; ++ks) {
                    const uint32_t kb = ks >> 2, sub = (ks & 3) * 32;
                    umma_bf16(d_tmem, umma_desc_sw128(k_addr + kb * kRegion + sub),
                              umma_desc_sw128(q_addr + kb * q_region + sub), idesc, ks > 0);
                }
                umma_commit(&bar.empty[st]);
                umma_commit(&bar.tfull[buf]);
            }
        }
    } else if (warp >= 4) {
        const int grp = (warp - 4) >> 2, quarter = warp & 3;
        const int L = quarter * 32 + lane;
        const float c = s.scale_log2;
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + grp * buf_cols;
        for (int t = grp; t < n_tiles; t += 2) {
            bool ok = mbar_wait(&bar.tfull[grp], (t >> 1) & 1, &abort_s);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            int cg = 0;
            for (; cg + 32 <= a.r16; cg += 32) {
                float v[32];
                tmem_ld32(taddr + cg, v);
#pragma unroll
                for (int x = 0; x < 32; x += 4) {
                    const float4 nl = *reinterpret_cast<const float4 *>(&neg_lse2[cg + x]);
                    a0 += fast_exp2(fmaf(v[x], c, nl.x));
                    a1 += fast_exp2(fmaf(v[x + 1], c, nl.y));
                    a2 += fast_exp2(fmaf(v[x + 2], c, nl.z));
                    a3 += fast_exp2(fmaf(v[x + 3], c, nl.w));
                }
            }
            if (cg < a.r16) {
                float v[16];
                tmem_ld16(taddr + cg, v);
#pragma unroll
                for (int x = 0; x < 16; x += 4) {
                    const float4 nl = *reinterpret_cast<const float4 *>(&neg_lse2[cg + x]);
                    a0 += fast_exp2(fmaf(v[x], c, nl.x));
                    a1 += fast_exp2(fmaf(v[x + 1], c, nl.y));
                    a2 += fast_exp2(fmaf(v[x + 2], c, nl.z));
                    a3 += fast_exp2(fmaf(v[x + 3], c, nl.w));
                }
            }
            tc_fence_before_sync();
            mbar_arrive(&bar.tempty[grp]);
            const float tj = (a0 + a1) + (a2 + a3);
            const int j = j_begin + t * kTile + L;
            if (j < j_end) {
                t_chunk[j - j_begin] = tj;
                if (a.token_scores) a.token_scores[(size_t)unit * s.nr_max + j] = tj;
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (!abort_s) {
        // Eq. 3-4: the block's windows (its first key is a multiple of omega)
        const int w_begin = j_begin / s.omega;
        const int n_win = (j_end - j_begin + s.omega - 1) / s.omega;
        for (int lw = threadIdx.x; lw < n_win; lw += kThreads) {
            const int lo = lw * s.omega;
            const int size = min(s.omega, (j_end - j_begin) - lo);
            a.window_scores[(size_t)unit * s.kw_max + w_begin + lw] = pool_top_p(t_chunk + lo, size, s.p);
        }
    } else if (threadIdx.x == 0) {
        atomicOr(a.status, kStatusWaitExpired);
    }
    if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)a.tmem_cols);
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &qres) ==
                cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// Tensor map of the leader's keys: dimension 0 is the head dimension; token, head and batch follow in
// order of increasing stride.  Box = 64 elements x 128 tokens, 128-byte swizzle, zero fill.
bool make_key_tensor_map(const KShape &ks, const void *k, CUtensorMap *tmap, int slot[3])
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) {
        set_error_detail("cuTensorMapEncodeTiled is not available from the driver");
        return false;
    }
    struct Dim {
        unsigned long long size, stride;
        int which;
    } dims[3] = {
        {(unsigned long long)(ks.cu ? ks.total_rows : ks.max_seqlen), (unsigned long long)ks.st * 2ull, 0},
        {(unsigned long long)ks.hkv, (unsigned long long)ks.sh * 2ull, 1},
        {(unsigned long long)(ks.cu ? 1 : ks.batch), (unsigned long long)ks.sb * 2ull, 2},
    };
    // dimensions of size one carry no address information: place them last with a synthetic stride
    std::stable_sort(dims, dims + 3, [](const Dim &x, const Dim &y) {
        const bool x1 = x.size == 1, y1 = y.size == 1;
        if (x1 != y1) return y1;
        return !x1 && x.stride < y.stride;
    });
    unsigned long long running = (unsigned long long)ks.d * 2ull;
    cuuint64_t gdim[4] = {(cuuint64_t)ks.d, 0, 0, 0}, gstride[3];
    cuuint32_t box[4] = {64, 1, 1, 1}, estr[4] = {1, 1, 1, 1};
    for (int i = 0; i < 3; ++i) {
        if (dims[i].size == 1) dims[i].stride = running;
        if (dims[i].stride == 0 || dims[i].stride % 16 || dims[i].stride >= (1ull << 40) ||
            dims[i].size > 0xffffffffull) {
            set_error_detail("key layout cannot be described by a tensor map (dimension %d: size %llu, stride %llu bytes)",
                             dims[i].which, dims[i].size, dims[i].stride);
            return false;
        }
        gdim[i + 1] = dims[i].size;
        gstride[i] = dims[i].stride;
        if (dims[i].which == 0) box[i + 1] = kTile;
        slot[dims[i].which] = i + 1;
        const unsigned long long span = dims[i].stride * dims[i].size;
        if (span > running) running = span;
    }
    const CUresult r = enc(tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(k), gdim, gstride, box,
                           estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error_detail("cuTensorMapEncodeTiled failed with code %d", (int)r);
        return false;
    }
    return true;
}

int device_cc_major()
{
    static int major = -1;
    static std::once_flag once;
    std::call_once(once, [] {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) {
            (void)cudaGetLastError();
            return;
        }
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess) major = v;
    });
    return major;
}

}  // namespace

bool score_tc_supported(const KShape &ks, int dtype)
{
    return dtype == WKV_BF16 && (ks.d == 64 || ks.d == 128) && ks.R <= 256 && ks.omega <= kTcMaxWindow &&
           device_cc_major() == 10;
}

int launch_score_tc(const KShape &ks, const void *q, const void *k, float *window_scores, float *token_scores,
                    void *workspace, const Workspace &ws, cudaStream_t stream)
{
    if (ks.max_seqlen - ks.alpha <= 0) return WKV_OK;
    alignas(64) CUtensorMap tmap;
    int slot[3] = {1, 2, 3};
    if (!make_key_tensor_map(ks, k, &tmap, slot)) return WKV_ERR_UNSUPPORTED;

    TcArgs a;
    a.s = ks;
    a.stats = reinterpret_cast<float2 *>(static_cast<char *>(workspace) + ws.stats_off);
    a.window_scores = window_scores;
    a.token_scores = token_scores;
    a.status = reinterpret_cast<int *>(static_cast<char *>(workspace) + ws.status_off);
    a.n_stat_chunks = ws.n_stat_chunks;
    a.r_pad = ws.r_pad;
    const int units = ks.batch * ks.hkv;
    a.chunks_per_unit = tc_chunks_per_unit(units, ks.max_seqlen);
    a.kblocks = ks.d / 64;
    a.slot_tok = slot[0];
    a.slot_h = slot[1];
    a.slot_b = slot[2];
    a.r16 = (ks.R + 15) / 16 * 16;
    int cols = 32;
    while (cols < 2 * a.r16) cols <<= 1;
    a.tmem_cols = cols;

    const int mb = ks.R > 128 ? 2 : 1;
    const size_t stage_bytes = (size_t)kStages * a.kblocks * kRegion;
    const size_t smem1 = 1024 + (size_t)a.kblocks * mb * 128 * 128 + stage_bytes;
    const size_t smem2 = 2048 + (size_t)a.kblocks * a.r16 * 128 + stage_bytes;
    dim3 grid(a.chunks_per_unit, units);
    cudaError_t err;
    const __nv_bfloat16 *qp = static_cast<const __nv_bfloat16 *>(q);
    if (mb == 1) {
        err = cudaFuncSetAttribute(score_stats_tc<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1);
        if (err == cudaSuccess) score_stats_tc<1><<<grid, kThreads, smem1, stream>>>(tmap, a, qp);
    } else {
        err = cudaFuncSetAttribute(score_stats_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1);
        if (err == cudaSuccess) score_stats_tc<2><<<grid, kThreads, smem1, stream>>>(tmap, a, qp);
    }
    if (err == cudaSuccess) err = cudaGetLastError();
    if (err == cudaSuccess)
        err = cudaFuncSetAttribute(score_pool_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2);
    if (err == cudaSuccess) {
        score_pool_tc<<<grid, kThreads, smem2, stream>>>(tmap, a, qp);
        err = cudaGetLastError();
    }
    if (err != cudaSuccess) {
        set_error_detail("tensor-core score kernels: %s", cudaGetErrorString(err));
        return WKV_ERR_CUDA;
    }
    count_launches(2);
    return WKV_OK;
}

}  // namespace wkv
