// Tensor-core score kernel (tcgen05 + tensor memory + TMA) for bf16 inputs: Eq. 1-4 of the leader
// and, when asked, the budgeted selection, in ONE cooperative launch.
//
// The token score of Eq. 2, t_j = sum_i exp(s_ij) / Z_i, needs every row's softmax normaliser
// Z_i (a reduction over all keys) before any column sum can be finished, so the keys are swept
// twice; a block starts normalising a unit's keys once all chunks of that unit have delivered their
// sweep-1 statistics (a per-unit arrival count, no grid-wide barrier):
//   sweep 1  D[rows, keys] = Q K^T per 128-key tile with the observation rows on the tensor-memory
//            lanes: one thread owns one row and keeps its running (max, sum exp2) without any
//            cross-thread traffic (Eq. 1's normaliser, causal mask on the tiles that touch the
//            observation window).  K comes from HBM.
//   sweep 2  D[keys, rows] = K Q^T with the keys on the lanes: one thread owns one key and sums
//            exp2(x_ij - lse2_i) over the rows (Eq. 2); the block then pools its windows (Eq. 3-4).
//            The block re-reads the keys it streamed in sweep 1, now from L2.
//   select   the block of a unit's last chunk waits for the unit's other blocks and runs the selection.
// Units are taken in waves whose keys fit L2 together.  A work item is (unit, chunk of <= 17 key
// tiles); the persistent blocks (at most one per SM) take the items of a wave round-robin.
//
// Warp roles: warp 0 issues the TMA tile loads (4-stage ring), warp 1 issues the MMAs into four
// accumulator buffers of 128 columns in tensor memory, and four compute groups of four warps (one
// warp per 32-lane quarter of tensor memory) take the accumulators round-robin, each with its own
// buffer, 32 columns at a time.  With more than 128 observation rows (up to 256) every key tile
// gives two accumulators, one per 128-row block of Q, which go through the same buffers and groups; the four warps that share an SM sub-partition cover each other's load latency.  The
// contraction is the only tensor-core work; exponentials, sums and pooling are fp32 on the CUDA
// cores in a fixed order, so results are bit-identical from run to run.
//
// Every wait is bounded (mbarriers and the wait for a unit's statistics): on expiry the block sets bit 0 of the
// status word, drains its own TMA loads, frees its tensor memory and returns.
#include "tc_common.cuh"
#include "score_math.cuh"
#include "topk_block.cuh"
#include "wkv_internal.cuh"

#include <cuda.h>

#include <algorithm>
#include <mutex>
#include <type_traits>

namespace wkv {
namespace {

using namespace tc;

constexpr int kStages = 4;
constexpr int kEarlyTiles = 2;                           // key tiles requested ahead of the Q image at the start of an item
constexpr int kMaxGroups = 4;
__host__ __device__ constexpr int groups_for(int) { return 4; }
__host__ __device__ constexpr int block_threads(int mb) { return 64 + groups_for(mb) * 128; }
constexpr int kTile = kTcTileKeys;                       // keys per tile
constexpr int kRegion = kTile * 128;                     // bytes of one 64-column block of a key tile
constexpr int kChunkCap = kTcMaxChunkTiles * kTile + kTcMaxWindow;   // token scores a block may hold

struct TcArgs {
    KShape s;
    float2 *stats;          // [units][n_stat_chunks][r_pad]
    float *window_scores;
    float *token_scores;
    const float *lse_obs;   // [B, H_q, alpha] natural log of Eq. 1's normalisers from the caller, or null
    int *window_idx;        // fused selection when non-null
    int *kept_len;
    int *status;
    int *sync;
    int n_stat_chunks, r_pad;
    int chunks_per_unit, units_per_wave;
    int kblocks;            // head_dim / 64
    int slot_tok, slot_h, slot_b;   // which tensor-map coordinate (1..3) carries token / head / batch
    int r16;                // observation rows rounded up to a multiple of 16
};

__device__ __forceinline__ uint8_t *align_1024(uint8_t *p)
{
    return reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(p) + 1023u) & ~uintptr_t(1023u));
}

struct Barriers {
    uint64_t full[kStages];        // TMA -> MMA: the stage holds a key tile
    uint64_t empty[kStages];       // MMA -> TMA: the MMAs that read the stage have completed
    uint64_t tfull[kMaxGroups];    // MMA -> compute group: the accumulator buffer is complete
    uint64_t tempty[kMaxGroups];   // compute group -> MMA: the accumulator buffer has been read
};

__device__ __forceinline__ void init_barriers(Barriers &bar)
{
    for (int i = 0; i < kStages; ++i) {
        mbar_init(&bar.full[i], 1);
        mbar_init(&bar.empty[i], 1);
    }
    for (int i = 0; i < kMaxGroups; ++i) {
        mbar_init(&bar.tfull[i], 1);
        mbar_init(&bar.tempty[i], 4);      // one arrival per warp of the group
    }
    fence_barrier_init();
}

// A compute warp waits through its lane 0 only (fewer threads hammering the barrier word leaves the
// shared-memory / special-function issue queue to the real work); the result is broadcast.
__device__ __forceinline__ bool warp_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int lane)
{
    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar, parity, abort_flag) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
// every lane has finished reading the accumulator buffer: hand it back to the MMA warp
__device__ __forceinline__ void warp_release(uint64_t *bar, int lane)
{
    tc_fence_before_sync();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
}

// Hand-over between the sweeps, per unit (all blocks are resident: cooperative launch).  A block that
// has written the sweep-1 statistics of one chunk adds one to the unit's arrival word; a block about
// to normalise keys of the unit waits until all of the unit's chunks have arrived.  No block waits
// before it has finished all its sweep-1 work, so every wait ends.  In sweep 2 every block counts
// itself on the unit's ticket word when it is done; the block of the unit's last chunk waits for
// that count (every waiter of the unit is past its wait by then), clears both words for the next
// launch and selects.  Bounded: a warp that waits longer than two seconds gives up and sets the
// block's abort flag.
// geometry of one work item
struct Item {
    int unit, chunk, b, h;
    int n, n_r;
    long long off;
    int j_begin, j_end, n_tiles;
    int reuse;   // sweep 2: the stage ring still holds the item's last tiles from sweep 1
};
// Tile taken at step u of an item.  Sweep 1 and a sweep 2 that has to load everything go through the
// tiles in ascending order.  A block that scores the item it has just taken statistics of still holds
// that item's last kStages tiles in the ring, in ring order: it scores those first, without
// loading them again, and then walks down through the rest.
__device__ __forceinline__ int tile_at(const Item &im, int u)
{
    if (!im.reuse) return u;
    return u < kStages ? im.n_tiles - kStages + u : im.n_tiles - 1 - u;
}

// ---------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------
template <int MB>   // 128-row blocks of observation rows: 1 (R <= 128) or 2 (R <= 256)
// 18 warps put five on one SM sub-partition (16K registers): 96 registers per thread at most
__global__ void __launch_bounds__(block_threads(MB), 1)
score_windows_tc(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ TcArgs a,
                 const __nv_bfloat16 *__restrict__ q)
{
    constexpr int NG = groups_for(MB);
    constexpr int kThreads = block_threads(MB);
    constexpr int q_rows = MB * 128;
    constexpr int q_region = q_rows * 128;                // bytes of one 64-column block of the Q image
    // A key tile gives one accumulator of 128 columns per 128-row block of Q ("half" rh = 0, 1 with
    // two row blocks); accumulators are numbered v = tile * MB + rh across the block's whole tile
    // stream, and buffers and compute groups take them round-robin (v mod NG).  With two row blocks a
    // group therefore always works on the same half (NG is even).
    constexpr uint32_t buf_cols = 128;                    // accumulator buffer stride in tensor memory
    constexpr uint32_t tmem_cols = 512;
    static_assert(NG * buf_cols <= tmem_cols, "accumulator buffers exceed tensor memory");

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) Barriers bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ float2 part[NG][1][128];                    // sweep 1: a group's (max, sum) of the rows on its lanes
    __shared__ __align__(16) float neg_lse2_all[256];    // -log2 of the row normaliser; -inf for padding rows
    __shared__ float t_chunk[MB][kChunkCap];              // sweep 2: per half, the key's sum over that half's rows
    __shared__ TopkSmem topk_sm;

    const KShape &s = a.s;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int units = s.batch * s.hkv;
    const int cpu = a.chunks_per_unit;
    const float c = s.scale_log2;

    uint8_t *q_img = align_1024(smem_raw);
    uint8_t *k_stage0 = q_img + a.kblocks * q_region;
    const int stage_bytes = a.kblocks * kRegion;
    const int ksteps = s.d / 16;

    if (threadIdx.x == 0) {
        init_barriers(bar);
        abort_s = 0;
    }
    if (warp == 1) tmem_alloc(&tmem_base_s, tmem_cols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_s;
    if (warp == 0 && lane == 0) tma_prefetch_desc(&tmap);

    // Row layout of the Q image: image row r holds observation row (r mod Rp); with Rp < 128 the rows
    // repeat so that all 128 lanes work in sweep 1, each copy taking its own slice of a tile's columns.
    // Rows [0, r16) of the image are the B operand of sweep 2.
    const int Rp = MB == 2 ? 256 : (s.R <= 32 ? 32 : (s.R <= 64 ? 64 : 128));
    int q_unit_loaded = -1;
    uint32_t it = 0;            // key tiles this block has pushed through the pipeline so far
    uint32_t p_issued = 0;      // producer thread only: tiles whose loads have been issued
    int s1_unit = -1, s1_chunk = -1, s1_tiles = 0;   // the sweep-1 item whose last tiles the ring holds ...
    uint32_t s1_it = 0;                              // ... as long as `it` still has this value

    auto make_item = [&](int unit, int chunk, int review_only, Item &im) {
        im.unit = unit;
        im.chunk = chunk;
        im.b = unit / s.hkv;
        im.h = unit % s.hkv;
        if (s.cu) {
            const int lo = min(max(s.cu[im.b], 0), s.total_rows);
            im.n = min(min(max(s.cu[im.b + 1] - s.cu[im.b], 0), s.n_cap), s.total_rows - lo);
            im.off = lo;
        } else {
            im.n = s.max_seqlen;
            im.off = 0;
        }
        im.n_r = im.n - s.alpha;
        const int n_keys = review_only ? im.n_r : im.n;
        const int len = tc_chunk_len(n_keys > 0 ? n_keys : 1, cpu, review_only ? s.omega : 1);
        im.j_begin = chunk * len;
        im.j_end = min(n_keys, im.j_begin + len);
        im.n_tiles = im.j_end > im.j_begin ? (im.j_end - im.j_begin + kTile - 1) / kTile : 0;
        im.reuse = 0;
    };

    // Called by every warp except the producer; ends with a barrier among those warps.  Four loads
    // are in flight per thread.  The producer starts streaming key tiles once these small loads
    // have been ISSUED (go_producer): a tile burst issued first would sit in front of them in the
    // SM's memory pipeline for microseconds.
    constexpr int kLoaders = kThreads - 32;
    auto go_producer = [&]() { asm volatile("bar.arrive 2, %0;" ::"n"(kThreads) : "memory"); };
    auto load_q_image = [&](const Item &im, bool signal) {
        if (q_unit_loaded != im.unit) {
            const __nv_bfloat16 *q_unit = q + im.b * s.qsb + (long long)im.h * s.G * s.qsh;
            const int vshift = s.d == 128 ? 4 : 3;            // log2(16-byte vectors per row)
            const int total = q_rows << vshift;
            for (int base = threadIdx.x - 32; base < total; base += kLoaders * 4) {
                int4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int idx = base + u * kLoaders;
                    v[u] = make_int4(0, 0, 0, 0);
                    if (idx < total) {
                        const int rq = (idx >> vshift) % Rp, cc = idx & ((1 << vshift) - 1);
                        if (rq < s.R) {
                            const int g = rq / s.alpha, i = rq - g * s.alpha;
                            v[u] = __ldg(reinterpret_cast<const int4 *>(q_unit + g * s.qsh + i * s.qst + cc * 8));
                        }
                    }
                }
                if (signal && base == (int)threadIdx.x - 32) go_producer();
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int idx = base + u * kLoaders;
                    if (idx < total) {
                        const int r = idx >> vshift, cc = idx & ((1 << vshift) - 1);
                        *reinterpret_cast<int4 *>(q_img + (cc >> 3) * q_region + swz128_offset(r, cc & 7)) = v[u];
                    }
                }
            }
            if (signal && (int)threadIdx.x - 32 >= total) go_producer();   // a thread without a share of the image
            fence_proxy_async_smem();
        } else if (signal) {
            go_producer();
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kLoaders) : "memory");
    };

    // producer: the item's key tiles into the stage ring (the block-wide tile counter `it` keeps the phases)
    auto produce = [&](const Item &im, int t_begin, int t_end) {
        const int tok0 = (int)im.off + im.j_begin;
        const int bcoord = s.cu ? 0 : im.b;
        for (int t = t_begin; t < t_end; ++t) {
            const uint32_t g = it + t;
            const int st = g % kStages;
            if (im.reuse && t < kStages) {
                // the stage holds this tile already: complete the phase without a load
                mbar_arrive(&bar.full[st]);
                ++p_issued;
                continue;
            }
            if (g >= kStages && !mbar_wait(&bar.empty[st], ((g / kStages) - 1) & 1, &abort_s)) return;
            mbar_arrive_expect_tx(&bar.full[st], (uint32_t)stage_bytes);
            const int tok = tok0 + tile_at(im, t) * kTile;
            const int c1 = a.slot_tok == 1 ? tok : (a.slot_h == 1 ? im.h : bcoord);
            const int c2 = a.slot_tok == 2 ? tok : (a.slot_h == 2 ? im.h : bcoord);
            const int c3 = a.slot_tok == 3 ? tok : (a.slot_h == 3 ? im.h : bcoord);
            for (int kb = 0; kb < a.kblocks; ++kb)
                tma_load_4d(k_stage0 + st * stage_bytes + kb * kRegion, &tmap, &bar.full[st], kb * 64, c1, c2, c3);
            ++p_issued;
        }
    };

    // MMA issue for one item.  sweep 1: D[rows, keys] = Q K^T; sweep 2: D[keys, rows] = K Q^T; per key
    // tile one accumulator per 128-row block of Q.
    // One thread issues everything, so its instruction count per tile is on the critical path: the
    // matrix descriptors of Q and of stage 0 are built once, and every k-step only adds a
    // compile-time constant to the address field (the fields above it never change).
    const uint64_t q_desc0 = umma_desc_sw128(smem_u32(q_img));
    const uint64_t k_desc0 = umma_desc_sw128(smem_u32(k_stage0));
    auto issue_tile = [&](auto ksteps_tag, uint32_t d_tmem, uint64_t k_desc, uint64_t q_desc, uint32_t idesc,
                          bool sweep2) {
        constexpr int KSTEPS = decltype(ksteps_tag)::value;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            const uint32_t qo = (uint32_t)((ks >> 2) * q_region + (ks & 3) * 32) >> 4;
            const uint32_t ko = (uint32_t)((ks >> 2) * kRegion + (ks & 3) * 32) >> 4;
            if (sweep2) umma_bf16(d_tmem, k_desc + ko, q_desc + qo, idesc, ks > 0);
            else umma_bf16(d_tmem, q_desc + qo, k_desc + ko, idesc, ks > 0);
        }
    };
    auto issue_mma = [&](const Item &im, bool sweep2) {
        const uint32_t stage_step = (uint32_t)stage_bytes >> 4;
        for (int t = 0; t < im.n_tiles; ++t) {
            const uint32_t g = it + t;
            const int st = g % kStages;
            if (!mbar_wait(&bar.full[st], (g / kStages) & 1, &abort_s)) return;
            const uint64_t k_desc = k_desc0 + (uint64_t)(st * stage_step);
#pragma unroll
            for (int rh = 0; rh < MB; ++rh) {
                const uint32_t v = g * MB + rh;
                const int buf = v % NG;
                if (v >= NG && !mbar_wait(&bar.tempty[buf], ((v / NG) - 1) & 1, &abort_s)) return;
                tc_fence_after_sync();
                // sweep 2: the rows of this half are the N dimension (a multiple of 16)
                const int n_rows = rh == 0 ? min(a.r16, 128) : a.r16 - 128;
                const uint32_t idesc = sweep2 ? umma_idesc_bf16(128, n_rows) : umma_idesc_bf16(128, kTile);
                const uint64_t q_desc = q_desc0 + (uint64_t)((rh * kRegion) >> 4);
                const uint32_t d_tmem = tmem_base + buf * buf_cols;
                if (ksteps == 8) issue_tile(std::integral_constant<int, 8>{}, d_tmem, k_desc, q_desc, idesc, sweep2);
                else issue_tile(std::integral_constant<int, 4>{}, d_tmem, k_desc, q_desc, idesc, sweep2);
                umma_commit(&bar.tfull[buf]);
            }
            umma_commit(&bar.empty[st]);
        }
    };

    const int grp = warp >= 2 ? (warp - 2) >> 2 : 0, quarter = warp & 3;
    const int L = quarter * 32 + lane;
    const uint32_t taddr_grp = tmem_base + ((uint32_t)(quarter * 32) << 16) + grp * buf_cols;

    // sweep-1 compute: the row's partial (max, sum exp2) over the item's keys -> part[grp][.][L]
    auto compute_stats = [&](const Item &im) {
        const int ncols = MB == 2 ? kTile : Rp;             // columns of a tile this thread reduces
        const int col0 = MB == 2 ? 0 : (L / Rp) * Rp;       // warp-uniform: Rp is a multiple of 32
        const int nslot = ncols >> 5;                       // 32-column slots of an accumulator this thread reduces
        float m0 = -INFINITY, l0 = 0.f;
        int limit0;                                         // last key the thread's row may attend to
        {
            const int row = MB == 2 ? (grp & 1) * 128 + L : L % Rp;
            limit0 = row < s.R ? min(im.n_r + row % s.alpha, im.j_end - 1) : -1;
        }
        const uint32_t taddr = taddr_grp + col0;
        for (uint32_t v = it * MB; v < (it + im.n_tiles) * MB; ++v) {
            if ((int)(v % NG) != grp) continue;
            const int t = (int)(v / MB - it);
            if (!warp_wait(&bar.tfull[grp], (v / NG) & 1, &abort_s, lane)) break;
            tc_fence_after_sync();
            const int tile0 = im.j_begin + t * kTile;
            const int j0 = tile0 + col0;
            const bool fast = (tile0 + kTile - 1 <= im.n_r) && (tile0 + kTile - 1 < im.j_end);   // no masking
            for (int sl = 0; sl < nslot; ++sl) {
                float x[32];
                tmem_ld32(taddr + sl * 32, x);
                if (sl + 1 == nslot) warp_release(&bar.tempty[grp], lane);   // the buffer may be overwritten now
                stats_update(x, fast, j0 + sl * 32, limit0, c, m0, l0);
            }
        }
        part[grp][0][L] = make_float2(m0, l0);
    };

    // sweep-2 compute: token score of key L of every tile of the item -> t_chunk (and token_scores)
    auto compute_scores = [&](const Item &im) {
        // rows of the group's half: 32-row slices; a 16-row tail follows if their number has bit 4 set
        const int rh = MB == 2 ? (grp & 1) : 0;
        const int rows_h = rh == 0 ? min(a.r16, 128) : a.r16 - 128;
        const int n32 = rows_h >> 5;
        const bool tail = (rows_h & 16) != 0;
        const float *neg_lse2 = neg_lse2_all + rh * 128;
        for (uint32_t av = it * MB; av < (it + im.n_tiles) * MB; ++av) {
            if ((int)(av % NG) != grp) continue;
            const int t = (int)(av / MB - it);
            if (!warp_wait(&bar.tfull[grp], (av / NG) & 1, &abort_s, lane)) break;
            tc_fence_after_sync();
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            for (int sl = 0; sl < n32; ++sl) {
                float v[32];
                tmem_ld32(taddr_grp + sl * 32, v);
                if (sl + 1 == n32 && !tail) warp_release(&bar.tempty[grp], lane);   // the buffer may be overwritten now
                score_accumulate<32>(v, neg_lse2 + sl * 32, c, a0, a1, a2, a3);
            }
            if (tail) {
                float vt[16];
                tmem_ld16(taddr_grp + n32 * 32, vt);
                warp_release(&bar.tempty[grp], lane);
                score_accumulate<16>(vt, neg_lse2 + n32 * 32, c, a0, a1, a2, a3);
            }
            const float tj = (a0 + a1) + (a2 + a3);
            const int j = im.j_begin + tile_at(im, t) * kTile + L;
            if (j < im.j_end) {
                t_chunk[rh][j - im.j_begin] = tj;
                if (MB == 1 && a.token_scores) a.token_scores[(size_t)im.unit * s.nr_max + j] = tj;
            }
        }
    };

    const int n_waves = (units + a.units_per_wave - 1) / a.units_per_wave;
    for (int wave = 0; wave < n_waves && !abort_s; ++wave) {
        const int u0 = wave * a.units_per_wave;
        const int nu = min(a.units_per_wave, units - u0);
        const int n_items = nu * cpu;

        // ------------------------------------------------------------------ sweep 1
        // (not needed when the caller supplies the normalisers: sweep 2 then reads the keys from HBM)
        for (int item = blockIdx.x; item < n_items && !a.lse_obs; item += gridDim.x) {
            Item im;
            make_item(u0 + item / cpu, item % cpu, 0, im);
            float2 *out = a.stats + ((size_t)im.unit * a.n_stat_chunks + im.chunk) * a.r_pad;
            if (im.n_r <= 0 || im.n_tiles == 0) {
                for (int r = threadIdx.x; r < a.r_pad; r += kThreads) out[r] = make_float2(-INFINITY, 0.f);
                continue;
            }
            if (warp == 0) {
                // the first tiles leave before the loads of the Q image (they land while those are
                // being issued); the rest of the ring's burst follows once the Q loads are on their way
                const int early = min(kEarlyTiles, im.n_tiles);
                if (lane == 0) produce(im, 0, early);
                asm volatile("bar.sync 2, %0;" ::"n"(kThreads) : "memory");
                if (lane == 0) produce(im, early, im.n_tiles);
            } else {
                load_q_image(im, true);
                if (warp == 1) {
                    if (lane == 0) issue_mma(im, false);
                } else {
                    compute_stats(im);
                }
            }
            q_unit_loaded = im.unit;
            it += im.n_tiles;
            s1_unit = im.unit;
            s1_chunk = im.chunk;
            s1_tiles = im.n_tiles;
            s1_it = it;
            tc_fence_before_sync();
            __syncthreads();
            tc_fence_after_sync();
            if (abort_s) break;
            // combine the compute groups and the column slices of each row, in a fixed order
            const int copies = MB == 2 ? 1 : 128 / Rp;
            for (int r = threadIdx.x; r < a.r_pad; r += kThreads) {
                float2 res = make_float2(-INFINITY, 0.f);
                if (r < s.R) {
                    const int mb = MB == 2 ? r >> 7 : 0, base = MB == 2 ? (r & 127) : r;
                    // with two row blocks a row lives in the groups of its half (group index odd or even)
                    float M = -INFINITY;
                    for (int g = 0; g < NG; ++g)
                        for (int cp = 0; cp < copies; ++cp)
                            if (MB == 1 || (g & 1) == mb) M = fmaxf(M, part[g][0][base + cp * Rp].x);
                    float sum = 0.f;
                    for (int g = 0; g < NG; ++g)
                        for (int cp = 0; cp < copies; ++cp) {
                            const float2 p = part[g][0][base + cp * Rp];
                            if ((MB == 1 || (g & 1) == mb) && p.y > 0.f) sum += p.y * fast_exp2((p.x - M) * c);
                        }
                    res = make_float2(M * c, sum);
                }
                out[r] = res;
            }
            __syncthreads();   // `part` is rewritten by the next item
            // release: cumulative over what the block wrote before the barrier above
            if (threadIdx.x == 0) red_release_gpu_add(a.sync + kSyncTickets + kSyncWordsPerUnit * im.unit + 1, 1);
        }
        if (abort_s) break;

        // ------------------------------------------------------------------ sweep 2 (+ selection)
        for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
            Item im;
            make_item(u0 + item / cpu, item % cpu, 1, im);
            const int kw = num_windows(im.n, s.alpha, s.omega);
            // read now, needed only by the block that selects: the load is long done by then
            const int budget = a.window_idx ? (s.budgets ? __ldg(s.budgets + im.b) : s.budget) : 0;
            if (im.n_r <= 0 || im.n_tiles == 0) {
                // a unit without review context still gets its (empty) selection, from its first item
                if (a.window_idx && im.n_r <= 0 && im.chunk == 0) {
                    select_topk_block<kThreads>(topk_sm, a.window_scores + (size_t)im.unit * s.kw_max, 0, 0, s.k_max,
                                                a.window_idx + (size_t)im.unit * s.k_max, a.kept_len + im.unit,
                                                im.n, s.alpha, s.omega);
                    __syncthreads();
                }
                continue;
            }
            const int len1 = tc_chunk_len(im.n, cpu, 1);
            im.reuse = im.unit == s1_unit && im.chunk == s1_chunk && it == s1_it && im.n_tiles == s1_tiles &&
                       im.n_tiles >= kStages && im.chunk * len1 == im.j_begin;
            if (warp == 0) {
                // ahead of the small loads of this item: the tiles the ring still holds (no traffic), or,
                // when this is the only sweep, the first tiles from HBM as in sweep 1
                const int ahead = im.reuse ? kStages : (a.lse_obs ? min(kEarlyTiles, im.n_tiles) : 0);
                if (lane == 0) produce(im, 0, ahead);
                asm volatile("bar.sync 2, %0;" ::"n"(kThreads) : "memory");
                if (lane == 0) produce(im, ahead, im.n_tiles);
            } else {
                load_q_image(im, false);
                if (warp == 1) {
                    // the MMAs do not need the normalisers: the first accumulators fill while the
                    // compute warps merge the statistics
                    go_producer();
                    if (lane == 0) issue_mma(im, true);
                } else {
                // Eq. 1's normaliser of every row: merge the partial statistics of the unit's chunks.
                // kMergers threads share a row (each takes every kMergers-th chunk), then one of them
                // merges their results; both steps in a fixed order.
                constexpr int kComputeThreads = kThreads - 64;
                constexpr int kMergers = kComputeThreads / q_rows;
                float2 *merged = &part[0][0][0];
                const int tl = threadIdx.x - 64;
                if (a.lse_obs) {
                    // the caller's normalisers, to base 2; row r = (query head g of the group, position i)
                    if (tl < 256) {
                        float v = -INFINITY;
                        if (tl < s.R) {
                            const int g = tl / s.alpha, i = tl - g * s.alpha;
                            v = -1.4426950408889634f *
                                __ldg(a.lse_obs + ((size_t)im.b * s.hq + (size_t)im.h * s.G + g) * s.alpha + i);
                        }
                        neg_lse2_all[tl] = v;
                    }
                    go_producer();
                    asm volatile("bar.sync 3, %0;" ::"n"(kComputeThreads) : "memory");
                    compute_scores(im);
                } else {
                const int used1 = (im.n + len1 - 1) / len1;   // chunks of the unit that hold keys in sweep 1
                const bool arrived =
                    warp_wait_arrivals(a.sync + kSyncTickets + kSyncWordsPerUnit * im.unit + 1, used1, &abort_s, lane);
                if (tl < kMergers * q_rows && arrived) {
                    const int r = tl % q_rows, mp = tl / q_rows;
                    float M = -INFINITY, sum = 0.f;
                    const int used = r < s.R ? used1 : 0;
                    const float2 *st = a.stats + (size_t)im.unit * a.n_stat_chunks * a.r_pad + r;
                    for (int c0 = mp; c0 < used || c0 == mp; c0 += 8 * kMergers) {
                        float2 p[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int cidx = c0 + u * kMergers;
                            p[u] = cidx < used ? __ldcg(st + (size_t)cidx * a.r_pad) : make_float2(-INFINITY, 0.f);
                        }
                        if (c0 == mp) go_producer();   // this thread's first loads are on their way
                        float Mn = M;
#pragma unroll
                        for (int u = 0; u < 8; ++u) Mn = fmaxf(Mn, p[u].x);
                        if (Mn > -INFINITY) {
                            sum *= fast_exp2(M - Mn);
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                if (p[u].y > 0.f) sum += p[u].y * fast_exp2(p[u].x - Mn);
                            M = Mn;
                        }
                    }
                    merged[mp * q_rows + r] = make_float2(M, sum);
                } else {
                    go_producer();
                }
                asm volatile("bar.sync 3, %0;" ::"n"(kComputeThreads) : "memory");
                if (tl < 256) {
                    float v = -INFINITY;
                    if (tl < s.R) {
                        float M = -INFINITY, sum = 0.f;
#pragma unroll
                        for (int mp = 0; mp < kMergers; ++mp) {
                            const float2 p = merged[mp * q_rows + tl];
                            if (p.y > 0.f) {
                                const float Mn = fmaxf(M, p.x);
                                sum = sum * fast_exp2(M - Mn) + p.y * fast_exp2(p.x - Mn);
                                M = Mn;
                            }
                        }
                        if (sum > 0.f) v = -(M + log2f(sum));
                    }
                    neg_lse2_all[tl] = v;
                }
                asm volatile("bar.sync 3, %0;" ::"n"(kComputeThreads) : "memory");
                compute_scores(im);
                }
                }
            }
            q_unit_loaded = im.unit;
            it += im.n_tiles;
            tc_fence_before_sync();
            __syncthreads();
            tc_fence_after_sync();
            if (abort_s) break;
            float *t_item = &t_chunk[0][0];
            if (MB == 2) {
                // Eq. 2 sums over all rows: add the two halves' sums of every key
                for (int x = threadIdx.x; x < im.j_end - im.j_begin; x += kThreads) {
                    const float tj = t_chunk[0][x] + t_chunk[MB - 1][x];
                    t_item[x] = tj;
                    if (a.token_scores) a.token_scores[(size_t)im.unit * s.nr_max + im.j_begin + x] = tj;
                }
                __syncthreads();
            }
            // Eq. 3-4: the item's windows (its first key is a multiple of omega)
            {
                const int n_tok = im.j_end - im.j_begin;
                float *ws_out = a.window_scores + (size_t)im.unit * s.kw_max + im.j_begin / s.omega;
                const int n_win = (n_tok + s.omega - 1) / s.omega;
                if (s.omega == 16 || s.omega == 8 || s.omega == 32 || s.omega == 4) {
                    // consecutive windows go to different warps so that all four schedulers take part
                    for (int i = threadIdx.x; i < n_win; i += kThreads) {
                        const int lw = i;
                        const int lo = lw * s.omega, size = min(s.omega, n_tok - lo);
                        float r;
                        if (s.omega == 16) r = pool_window_sorted<16>(t_item + lo, size, s.p);
                        else if (s.omega == 8) r = pool_window_sorted<8>(t_item + lo, size, s.p);
                        else if (s.omega == 32) r = pool_window_sorted<32>(t_item + lo, size, s.p);
                        else r = pool_window_sorted<4>(t_item + lo, size, s.p);
                        ws_out[lw] = r;
                    }
                }
                else if (s.omega == 64 || s.omega == 128) {
                    // one warp per window
                    for (int lw = warp; lw < n_win; lw += kThreads / 32) {
                        const int lo = lw * s.omega, size = min(s.omega, n_tok - lo);
                        const float r = s.omega == 64 ? pool_window_warp<64>(t_item + lo, size, s.p, lane)
                                                      : pool_window_warp<128>(t_item + lo, size, s.p, lane);
                        if (lane == 0) ws_out[lw] = r;
                    }
                }
                else {
                    for (int lw = threadIdx.x; lw < n_win; lw += kThreads) {
                        const int lo = lw * s.omega;
                        ws_out[lw] = pool_top_p(t_item + lo, min(s.omega, n_tok - lo), s.p);
                    }
                }
            }
            const int len2 = tc_chunk_len(im.n_r, cpu, s.omega);
            const int used2 = (im.n_r + len2 - 1) / len2;   // chunks of the unit that hold keys in sweep 2
            // The block of the unit's last chunk selects for the unit (and clears the unit's words): that
            // chunk is usually a short one, so its block is done early and the selection does not sit
            // on the path of a block that the next wave is waiting for.  The other blocks only count
            // themselves, without waiting for an answer.
            int *ticket = a.sync + kSyncTickets + kSyncWordsPerUnit * im.unit;
            if (im.chunk != used2 - 1) {
                if (a.window_idx) {
                    __syncthreads();
                    // release, cumulative: publishes the window scores the whole block wrote
                    if (threadIdx.x == 0) red_release_gpu_add(ticket, 1);
                } else if (threadIdx.x == 0) {
                    atomicAdd(ticket, 1);
                }
            } else {
                __syncthreads();
                if (threadIdx.x == 0 && poll_until_at_least(ticket, used2 - 1, &abort_s)) {
                    atomicExch(ticket, 0);       // every other block of the unit is past its waits
                    atomicExch(ticket + 1, 0);
                }
                __syncthreads();
                if (a.window_idx && !abort_s) {
                    select_topk_block<kThreads>(topk_sm, a.window_scores + (size_t)im.unit * s.kw_max, kw,
                                                num_selected_capped(im.n, s.alpha, s.omega, budget, s.k_max), s.k_max,
                                                a.window_idx + (size_t)im.unit * s.k_max, a.kept_len + im.unit,
                                                im.n, s.alpha, s.omega);
                }
            }
            __syncthreads();   // t_chunk, neg_lse2 and the selection scratch are reused by the next item
        }
    }

    // ------------------------------------------------------------------ teardown
    __syncthreads();
    if (warp == 0 && lane == 0) {
        // nothing of this block may be in flight when it ends: the last MMAs must have released
        // their stages; after a failed wait, the loads already issued must still land
        for (uint32_t g = p_issued > kStages ? p_issued - kStages : 0; g < p_issued; ++g) {
            const int st = g % kStages;
            if (!mbar_wait(&bar.empty[st], (g / kStages) & 1, &abort_s)) {
                volatile int never = 0;
                mbar_wait(&bar.full[st], (g / kStages) & 1, &never);
            }
        }
        if (abort_s) atomicOr(a.status, kStatusWaitExpired);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);
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

// What the launcher needs to know about a device and its copy of the kernels, looked up on the first
// use of that device: kernel attributes (the shared-memory opt-in) belong to a device, so a process
// that drives several GPUs sets them on each.
struct DeviceInfo {
    bool known = false;
    int cc_major = -1;
    int sm_count = 0;
    int cooperative = 0;
    int blocks_per_sm[2] = {-1, -1};   // resident blocks of each instantiation at its largest footprint
};
std::mutex g_device_mutex;
DeviceInfo g_device_info[kMaxDevices];
// the current device's entry (callers hold no lock: entries are only ever filled in, under the mutex)
DeviceInfo *device_info()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return nullptr;
    }
    std::lock_guard<std::mutex> lock(g_device_mutex);
    DeviceInfo &info = g_device_info[dev];
    if (!info.known) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess) info.cc_major = v;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess) info.sm_count = v;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess) info.cooperative = v;
        (void)cudaGetLastError();
        info.known = true;
    }
    return &info;
}

size_t tc_smem_bytes(int kblocks, int mb)
{
    return 1024 + (size_t)kblocks * mb * 128 * 128 + (size_t)kStages * kblocks * kRegion;
}

}  // namespace

bool score_tc_supported(const KShape &ks, int dtype)
{
    const DeviceInfo *di = device_info();
    return di && dtype == WKV_BF16 && (ks.d == 64 || ks.d == 128) && ks.R <= 256 && ks.omega <= kTcMaxWindow &&
           di->cc_major == 10 && di->cooperative && di->sm_count > 0;
}

int launch_score_tc(const KShape &ks, const void *q, const void *k, float *window_scores, float *token_scores,
                    int *window_idx, int *kept_len, void *workspace, const Workspace &ws, cudaStream_t stream,
                    const float *lse_obs)
{
    alignas(64) CUtensorMap tmap;
    int slot[3] = {1, 2, 3};
    if (!make_key_tensor_map(ks, k, &tmap, slot)) return WKV_ERR_UNSUPPORTED;
    DeviceInfo *dip = device_info();
    if (!dip) {
        set_error_detail("no current CUDA device, or its ordinal is beyond %d", kMaxDevices - 1);
        return WKV_ERR_CUDA;
    }
    DeviceInfo &di = *dip;

    TcArgs a;
    a.s = ks;
    a.stats = reinterpret_cast<float2 *>(static_cast<char *>(workspace) + ws.stats_off);
    a.window_scores = window_scores;
    a.lse_obs = lse_obs;
    a.token_scores = token_scores;
    a.window_idx = window_idx;
    a.kept_len = kept_len;
    a.status = reinterpret_cast<int *>(static_cast<char *>(workspace) + ws.status_off);
    a.sync = reinterpret_cast<int *>(static_cast<char *>(workspace) + ws.sync_off);
    a.n_stat_chunks = ws.n_stat_chunks;
    a.r_pad = ws.r_pad;
    const int units = ks.batch * ks.hkv;
    const TcPlan plan = tc_plan(units, ks.max_seqlen, ks.d);
    a.chunks_per_unit = plan.chunks_per_unit;
    a.units_per_wave = plan.units_per_wave;
    a.kblocks = ks.d / 64;
    a.slot_tok = slot[0];
    a.slot_h = slot[1];
    a.slot_b = slot[2];
    a.r16 = (ks.R + 15) / 16 * 16;

    const int mb = ks.R > 128 ? 2 : 1;
    const int threads = block_threads(mb);
    const size_t smem = tc_smem_bytes(a.kblocks, mb);
    const void *fn = mb == 1 ? reinterpret_cast<const void *>(score_windows_tc<1>)
                             : reinterpret_cast<const void *>(score_windows_tc<2>);
    cudaError_t err = cudaSuccess;
    std::unique_lock<std::mutex> setup_lock(g_device_mutex);
    if (di.blocks_per_sm[mb - 1] < 0) {
        // once per device and instantiation: allow its largest shared-memory request (head_dim 128) and ask how
        // many of its blocks an SM holds at that size
        const size_t smem_max = tc_smem_bytes(2, mb);
        err = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
        if (err == cudaSuccess)
            err = cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        int occ = 0;
        if (err == cudaSuccess) err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, fn, threads, smem_max);
        if (err == cudaSuccess) {
            if (occ < 1) {
                cudaFuncAttributes fa;
                (void)cudaFuncGetAttributes(&fa, fn);
                set_error_detail("tensor-core score kernel does not fit an SM (%d threads, %d registers, %zu + %zu bytes "
                                 "of shared memory)", threads, fa.numRegs, smem_max, fa.sharedSizeBytes);
                return WKV_ERR_CUDA;
            }
            di.blocks_per_sm[mb - 1] = occ;
        }
    }
    setup_lock.unlock();
    // persistent blocks, one per SM at most; every block of a cooperative launch is resident, which
    // the hand-over of the statistics between the sweeps relies on
    int grid = plan.units_per_wave * plan.chunks_per_unit;
    if (grid > di.sm_count) grid = di.sm_count;
    const __nv_bfloat16 *qp = static_cast<const __nv_bfloat16 *>(q);
    if (err == cudaSuccess) {
        void *params[3] = {&tmap, &a, &qp};
        err = cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(threads), params, smem, stream);
    }
    if (err != cudaSuccess) {
        set_error_detail("tensor-core score kernel (grid %d x %d threads, %zu bytes of shared memory): %s", grid,
                         threads, smem, cudaGetErrorString(err));
        return WKV_ERR_CUDA;
    }
    count_launches(1);
    return WKV_OK;
}

}  // namespace wkv
