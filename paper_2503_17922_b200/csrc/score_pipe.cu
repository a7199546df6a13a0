// Pipelined group kernel (tcgen05 + tensor memory + TMA) for bf16 inputs with at most 128 observation
// rows per unit: Eq. 1-4 of the leader, the budgeted selection and, when asked, the shared-index
// gather of every layer of the group (section 2.2.2), in ONE cooperative launch.
//
// The arithmetic is that of score_tc.cu (two sweeps over the keys: Eq. 1's row statistics with the
// observation rows on the tensor-memory lanes, then Eq. 2's normalised column sums with the keys on
// the lanes, pooling by sorting network, selection by the block of a unit's last chunk).  What differs
// is the schedule:
//   * The units are taken in waves, and the statistics sweep runs ONE WAVE AHEAD of the scoring
//     sweep: a block's work is  s1(wave 0), s1(wave 1), s2(wave 0), s1(wave 2), s2(wave 1), ...
//     By the time a block normalises a unit, the statistics of that unit's other chunks were
//     published a whole sweep ago, so the hand-over between blocks costs no waiting, and while wave w
//     is being scored the rows of wave w-1, whose selection is already known, are being gathered.
//   * Every role runs through the block's whole list of work items on its own and meets the others
//     only through mbarriers: warp 0 streams key tiles (and the Q images) by TMA, warp 1 issues the
//     MMAs, sixteen compute warps take the accumulators, and none of them stops at an item boundary
//     for the others (the tile ring and the accumulator buffers are filled across items).
//   * Two copy warps gather: as soon as a unit's selection is published they move its retained
//     windows of every layer's K and V with bulk asynchronous copies (global -> shared -> global,
//     4 KB slots, L2 evict-first so that the keys of the wave still to be scored stay in L2).  Jobs are
//     handed out through one counter per unit, so when the scoring is over the producer warp joins in
//     with the idle tile ring as 32 more slots and the tail of the gather runs at the copy rate.
// The Q image of an item's unit is fetched by TMA when the producer reaches the item (32 KB out of L2,
// behind the accumulators the compute warps still have to work through).
// The per-chunk row statistics travel between blocks as self-validating 8-byte entries (the low
// mantissa bit of the sum marks an entry as written; the area is zero between launches), so that
// publishing them needs no fence and reading them no counter.
//
// Every wait is bounded (mbarriers, arrival counts, selection flags): on expiry the block sets bit 0
// of the status word, lets its own asynchronous copies land, frees its tensor memory and returns.
#include "score_math.cuh"
#include "tc_common.cuh"
#include "topk_block.cuh"
#include "wkv_internal.cuh"

#include <cuda.h>

#include <algorithm>
#include <mutex>

namespace wkv {
namespace {

using namespace tc;

constexpr int kStages = 4;                               // key tiles in flight
constexpr int kBufs = 4;                                 // accumulator buffers of 128 columns
constexpr int kTile = kTcTileKeys;
constexpr int kRegion = kTile * 128;                     // bytes of one 64-column block of a key tile
constexpr int kQRows = 128;                              // rows of a Q image
constexpr int kQRegion = kQRows * 128;                   // bytes of one 64-column block of a Q image
constexpr int kChunkCap = kTcMaxChunkTiles * kTile + kTcMaxWindow;
constexpr int kComputeWarps = 16;
constexpr int kComputeThreads = kComputeWarps * 32;      // threads 64 .. 575
constexpr int kCopyWarps = 2;
constexpr int kThreads = 64 + kComputeThreads + kCopyWarps * 32;
constexpr int kCopySlotBytes = 4096;
constexpr int kCopySlots = 5;                            // per copy warp
constexpr int kTailSlotsMax = 32;                        // slots the producer warp carves out of the tile ring
constexpr int kBarCompute = 3;                           // named barrier of the compute warps

struct PipeArgs {
    KShape s;
    unsigned long long *pstats;   // [units][n_stat_chunks][128] self-validating (max, sum) entries, zero between launches
    float *window_scores;
    float *token_scores;
    const float *lse_obs;
    int *window_idx;        // selection when non-null
    int *kept_len;
    int *status;
    int *sync;
    int n_stat_chunks;
    int chunks_per_unit, units_per_wave, n_waves, skew;
    int kblocks;            // head_dim / 64
    int slot_tok, slot_h, slot_b;
    int r16, Rp, q_copies;
    // gather (n_tensors == 0: none)
    int n_tensors;
    int keep_capacity;
    const int *cu_out;
    int row_bytes;
    long long src_row_stride;   // bytes between consecutive source rows of a unit
    int rows_per_job, subs_per_window, obs_slots;
    LayerTable tab;
};

// words of the synchronisation area used here (see wkv_internal.cuh for the per-unit words)
constexpr int kSyncCopiersDone = 1;

__device__ __forceinline__ uint8_t *align_1024(uint8_t *p)
{
    return reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(p) + 1023u) & ~uintptr_t(1023u));
}

struct PipeBarriers {
    uint64_t full[kStages], empty[kStages];
    uint64_t tfull[kBufs], tempty[kBufs];
    uint64_t qfull, qfree;
    uint64_t copy[kCopyWarps][kCopySlots];
    uint64_t tail[kTailSlotsMax];
};

__device__ __forceinline__ bool warp_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int lane)
{
    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar, parity, abort_flag) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
__device__ __forceinline__ void warp_release(uint64_t *bar, int lane)
{
    tc_fence_before_sync();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
}
__device__ __forceinline__ void compute_sync()
{
    asm volatile("bar.sync %0, %1;" ::"n"(kBarCompute), "n"(kComputeThreads) : "memory");
}
__device__ __forceinline__ void st_release_gpu(int *p, int v)
{
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// ---- self-validating statistics entries ----------------------------------------------------------
// One 8-byte word per (unit, chunk, row): the row's maximum (times log2(e)/sqrt(d)) in the low half and
// its sum of exponentials in the high half, with the lowest mantissa bit of the sum forced to one so
// that a written entry is never all zero (an empty row's sum 0 becomes the smallest denormal).  The
// reader clears that bit again: the sum loses at most one unit in the last place.  Written and read
// with single 64-bit accesses, so an entry is seen whole or not at all.
__device__ __forceinline__ unsigned long long stat_pack(float m, float sum)
{
    const unsigned hi = sum == 0.f ? 1u : (__float_as_uint(sum) | 1u);
    return ((unsigned long long)hi << 32) | (unsigned long long)__float_as_uint(m);
}
__device__ __forceinline__ bool stat_unpack(unsigned long long w, float2 &out)
{
    const unsigned hi = (unsigned)(w >> 32);
    out.x = __uint_as_float((unsigned)w);
    out.y = __uint_as_float(hi & ~1u);
    return hi != 0u;
}
__device__ __forceinline__ void st_relaxed_gpu_u64(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_relaxed_gpu_u64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// ---- bulk asynchronous copies (no multicast) ----------------------------------------------------
__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// global -> this block's shared memory; 16-byte aligned addresses, size a multiple of 16
__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar, uint64_t pol)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 :
                 : "r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(pol)
                 : "memory");
}
__device__ __forceinline__ void bulk_store(void *gdst, const void *smem_src, uint32_t bytes, uint64_t pol)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                 :
                 : "l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes), "l"(pol)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ---- the block's list of work items ------------------------------------------------------------
// phase 0: statistics sweep (all keys the rows may attend to), phase 1: scoring sweep (review keys)
struct Entry {
    int phase, wave, unit, chunk, b, h;
    int n, n_r;
    long long off;
    int j_begin, j_end, n_tiles;
};
struct Cursor {
    int step, phase, j;
};
__device__ __forceinline__ void cursor_init(Cursor &c)
{
    c.step = 0;
    c.phase = 0;
    c.j = 0;
}
// Every thread of the block walks the same list, computed from the launch arguments and the block
// index alone: step s holds the block's statistics items of wave s, then its scoring items of wave
// s - skew.
__device__ __forceinline__ bool next_entry(const PipeArgs &a, Cursor &c, Entry &e)
{
    const KShape &s = a.s;
    const int units = s.batch * s.hkv;
    const int n_steps = a.n_waves + a.skew;
    for (;;) {
        if (c.step >= n_steps) return false;
        const int wave = c.phase == 0 ? c.step : c.step - a.skew;
        const bool live = c.phase == 0 ? (!a.lse_obs && wave < a.n_waves) : (wave >= 0 && wave < a.n_waves);
        if (live) {
            const int u0 = wave * a.units_per_wave;
            const int nu = min(a.units_per_wave, units - u0);
            const int item = (int)blockIdx.x + c.j * (int)gridDim.x;
            if (item < nu * a.chunks_per_unit) {
                ++c.j;
                e.phase = c.phase;
                e.wave = wave;
                e.unit = u0 + item / a.chunks_per_unit;
                e.chunk = item % a.chunks_per_unit;
                e.b = e.unit / s.hkv;
                e.h = e.unit % s.hkv;
                if (s.cu) {
                    const int lo = min(max(s.cu[e.b], 0), s.total_rows);
                    e.n = min(min(max(s.cu[e.b + 1] - s.cu[e.b], 0), s.n_cap), s.total_rows - lo);
                    e.off = lo;
                } else {
                    e.n = s.max_seqlen;
                    e.off = 0;
                }
                e.n_r = e.n - s.alpha;
                const int n_keys = e.phase ? e.n_r : e.n;
                const int len = tc_chunk_len(n_keys > 0 ? n_keys : 1, a.chunks_per_unit, e.phase ? s.omega : 1);
                e.j_begin = e.chunk * len;
                e.j_end = min(n_keys, e.j_begin + len);
                e.n_tiles = (e.n_r > 0 && e.j_end > e.j_begin) ? (e.j_end - e.j_begin + kTile - 1) / kTile : 0;
                return true;
            }
        }
        if (c.phase == 0) {
            c.phase = 1;
            c.j = 0;
        } else {
            c.phase = 0;
            c.j = 0;
            ++c.step;
        }
    }
}

// Which unit's queries the Q image holds; producer and MMA warp keep identical copies of this state
// by walking the same list, so both know when the image is (re)loaded.
struct QState {
    int unit;
    uint32_t loads;      // images loaded so far
    uint32_t frees;      // hand-backs of the image (MMA warp -> producer) so far
};

// ---------------------------------------------------------------------------------------------
// gather by bulk copies: one warp, lane l drives slot l
// ---------------------------------------------------------------------------------------------
// Goes through the units in order; for each waits until its selection has been published, then takes
// batches of jobs from the unit's counter until none are left.  A job is (tensor, window slot,
// sub-range of at most rows_per_job rows): loaded into the lane's slot, then stored from there.
// `phase` holds one parity bit per lane's barrier.  Returns false after an expired wait.
__device__ bool copy_units(const PipeArgs &a, uint8_t *slots, uint64_t *bars, int n_slots, uint32_t &phase,
                           volatile int *abort_flag, int lane)
{
    const KShape &s = a.s;
    const uint64_t pol = l2_evict_first_policy();
    const int units = s.batch * s.hkv;
    const int elem_bytes = a.row_bytes / s.d;
    uint8_t *my_slot = slots + (size_t)lane * kCopySlotBytes;
    for (int unit = 0; unit < units; ++unit) {
        int *flag = a.sync + kSyncTickets + kSyncWordsPerUnit * unit + 2;
        int *ctr = flag + 1;
        int ok = 1;
        if (lane == 0) ok = poll_until_at_least(flag, 1, abort_flag, 400) ? 1 : 0;
        if (!__shfl_sync(0xffffffffu, ok, 0)) return false;
        const int b = unit / s.hkv, h = unit % s.hkv;
        const SeqInfo si = seq_info(s, b);
        const int n = si.n;
        const int n_r = n > s.alpha ? n - s.alpha : 0;
        const int kw = num_windows(n, s.alpha, s.omega);
        const int k = num_selected_capped(n, s.alpha, s.omega, si.budget, s.k_max);
        const int *idx = a.window_idx + (size_t)unit * s.k_max;
        int review_rows = k * s.omega;
        if (k > 0 && __ldcg(idx + k - 1) == kw - 1) review_rows -= kw * s.omega - n_r;
        const int obs_rows = n - n_r;
        const int n_slots_u = k + a.obs_slots;
        const int n_jobs = a.n_tensors * n_slots_u * a.subs_per_window;
        const long long src_off = (si.off * s.st + b * s.sb + h * s.sh) * (long long)elem_bytes;
        long long dst_off, dst_row_stride;
        if (a.cu_out) {
            dst_off = ((long long)a.cu_out[b] * s.hkv + h) * a.row_bytes;
            dst_row_stride = (long long)s.hkv * a.row_bytes;
        } else {
            dst_off = (long long)unit * a.keep_capacity * a.row_bytes;
            dst_row_stride = a.row_bytes;
        }
        const bool contiguous = a.src_row_stride == a.row_bytes && dst_row_stride == a.row_bytes;
        for (;;) {
            int base = 0;
            if (lane == 0) base = atomicAdd(ctr, n_slots);
            base = __shfl_sync(0xffffffffu, base, 0);
            if (base >= n_jobs) break;
            const int j = base + lane;
            bool active = lane < n_slots && j < n_jobs;
            const uint8_t *src = nullptr;
            uint8_t *dst = nullptr;
            int rows = 0;
            if (active) {
                const int sub = j % a.subs_per_window;
                const int w = (j / a.subs_per_window) % n_slots_u;
                const int tensor = j / (a.subs_per_window * n_slots_u);
                int src_row0, dst_row0, n_rows;
                if (w < k) {
                    // an entry that is no window of this sequence is skipped, never followed
                    const int wi = __ldcg(idx + w);
                    src_row0 = wi * s.omega;
                    n_rows = (wi < 0 || wi >= kw) ? 0 : min(s.omega, n_r - src_row0);
                    dst_row0 = w * s.omega;
                } else {
                    const int o = (w - k) * s.omega;
                    src_row0 = n_r + o;
                    n_rows = min(s.omega, obs_rows - o);
                    dst_row0 = review_rows + o;
                }
                const int r0 = sub * a.rows_per_job;
                rows = min(a.rows_per_job, n_rows - r0);
                if (!a.cu_out && dst_row0 + r0 + rows > a.keep_capacity) rows = 0;
                active = rows > 0;
                src = static_cast<const uint8_t *>(a.tab.src[tensor]) + src_off + (long long)(src_row0 + r0) * a.src_row_stride;
                dst = static_cast<uint8_t *>(a.tab.dst[tensor]) + dst_off + (long long)(dst_row0 + r0) * dst_row_stride;
            }
            bool landed = true;
            if (active) {
                mbar_arrive_expect_tx(&bars[lane], (uint32_t)(rows * a.row_bytes));
                if (contiguous) {
                    bulk_load(my_slot, src, (uint32_t)(rows * a.row_bytes), &bars[lane], pol);
                } else {
                    for (int r = 0; r < rows; ++r)
                        bulk_load(my_slot + r * a.row_bytes, src + (long long)r * a.src_row_stride, (uint32_t)a.row_bytes,
                                  &bars[lane], pol);
                }
                landed = mbar_wait(&bars[lane], (phase >> lane) & 1u, abort_flag);
                if (!landed) {
                    // the copy is still on its way into this block's shared memory: let it land
                    volatile int never = 0;
                    mbar_wait(&bars[lane], (phase >> lane) & 1u, &never);
                } else {
                    fence_proxy_async_smem();
                    if (contiguous) {
                        bulk_store(dst, my_slot, (uint32_t)(rows * a.row_bytes), pol);
                    } else {
                        for (int r = 0; r < rows; ++r)
                            bulk_store(dst + (long long)r * dst_row_stride, my_slot + r * a.row_bytes, (uint32_t)a.row_bytes, pol);
                    }
                    bulk_commit();
                }
                phase ^= 1u << lane;
            }
            bulk_wait_read_all();
            if (!__all_sync(0xffffffffu, landed)) return false;
        }
    }
    return true;
}

// Every copier warp of the grid (two per block and each block's producer warp) reports here when it has
// been through all units; the last one clears the flags and job counters for the next launch.
__device__ void copiers_done(const PipeArgs &a, int lane)
{
    bulk_wait_all();
    if (lane == 0) {
        __threadfence();
        const int total = (int)gridDim.x * (kCopyWarps + 1);
        if (atomicAdd(a.sync + kSyncCopiersDone, 1) == total - 1) {
            const int units = a.s.batch * a.s.hkv;
            for (int u = 0; u < units; ++u) {
                a.sync[kSyncTickets + kSyncWordsPerUnit * u + 2] = 0;
                a.sync[kSyncTickets + kSyncWordsPerUnit * u + 3] = 0;
            }
            a.sync[kSyncCopiersDone] = 0;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1)
group_pipeline_tc(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap qmap,
                  const __grid_constant__ PipeArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) PipeBarriers bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ float2 part[kBufs][128];                  // a compute group's (max, sum) of the rows on its lanes
    __shared__ __align__(16) float neg_lse2[128];        // -log2 of the row normaliser; -inf for padding rows
    __shared__ float t_chunk[kChunkCap];                 // token scores of the item being scored
    __shared__ TopkSmem topk_sm;

    const KShape &s = a.s;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cpu = a.chunks_per_unit;
    const float c = s.scale_log2;
    constexpr uint32_t tmem_cols = 512;

    const int q_img_bytes = a.kblocks * kQRegion;
    const int stage_bytes = a.kblocks * kRegion;
    uint8_t *q_img0 = align_1024(smem_raw);
    uint8_t *k_stage0 = q_img0 + q_img_bytes;
    uint8_t *copy_ring = k_stage0 + kStages * stage_bytes;
    const int ksteps = s.d / 16;
    const bool gathers = a.n_tensors > 0 && a.window_idx != nullptr;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&bar.full[i], 1);
            mbar_init(&bar.empty[i], 1);
        }
        for (int i = 0; i < kBufs; ++i) {
            mbar_init(&bar.tfull[i], 1);
            mbar_init(&bar.tempty[i], 4);     // one arrival per warp of the group
        }
        mbar_init(&bar.qfull, 1);
        mbar_init(&bar.qfree, 1);
        for (int i = 0; i < kCopyWarps * kCopySlots; ++i) mbar_init(&bar.copy[0][0] + i, 1);
        for (int i = 0; i < kTailSlotsMax; ++i) mbar_init(&bar.tail[i], 1);
        fence_barrier_init();
        abort_s = 0;
    }
    if (warp == 1) tmem_alloc(&tmem_base_s, tmem_cols);
    // rows of the Q image that no load ever writes (padding up to the image height) must read as zero
    for (int i = threadIdx.x; i < q_img_bytes / 16; i += kThreads)
        reinterpret_cast<int4 *>(q_img0)[i] = make_int4(0, 0, 0, 0);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_s;

    if (warp == 0) {
        // ================================================================== producer
        uint32_t issued = 0;          // key tiles requested so far
        QState qs = {-1, 0, 0};
        if (lane == 0) {
            tma_prefetch_desc(&kmap);
            tma_prefetch_desc(&qmap);
            Cursor cur;
            cursor_init(cur);
            Entry e;
            bool ok = true;
            while (ok && next_entry(a, cur, e)) {
                if (e.n_tiles == 0) continue;
                if (qs.unit != e.unit) {
                    // the MMAs that read the old image must have completed (signalled by the MMA warp
                    // when it reaches this item)
                    if (qs.unit != -1) {
                        ok = mbar_wait(&bar.qfree, qs.frees & 1u, &abort_s);
                        ++qs.frees;
                        if (!ok) break;
                    }
                    mbar_arrive_expect_tx(&bar.qfull, (uint32_t)(a.q_copies * a.kblocks * s.R * 128));
                    for (int cp = 0; cp < a.q_copies; ++cp)
                        for (int kb = 0; kb < a.kblocks; ++kb)
                            tma_load_4d(q_img0 + kb * kQRegion + cp * a.Rp * 128, &qmap, &bar.qfull, kb * 64, 0,
                                        e.h * s.G, e.b);
                    qs.unit = e.unit;
                    ++qs.loads;
                }
                const int tok0 = (int)e.off + e.j_begin;
                const int bcoord = s.cu ? 0 : e.b;
                for (int t = 0; t < e.n_tiles; ++t) {
                    const uint32_t g = issued;
                    const int st = g % kStages;
                    if (g >= kStages && !mbar_wait(&bar.empty[st], ((g / kStages) - 1) & 1, &abort_s)) {
                        ok = false;
                        break;
                    }
                    mbar_arrive_expect_tx(&bar.full[st], (uint32_t)stage_bytes);
                    const int tok = tok0 + t * kTile;
                    const int c1 = a.slot_tok == 1 ? tok : (a.slot_h == 1 ? e.h : bcoord);
                    const int c2 = a.slot_tok == 2 ? tok : (a.slot_h == 2 ? e.h : bcoord);
                    const int c3 = a.slot_tok == 3 ? tok : (a.slot_h == 3 ? e.h : bcoord);
                    for (int kb = 0; kb < a.kblocks; ++kb)
                        tma_load_4d(k_stage0 + st * stage_bytes + kb * kRegion, &kmap, &bar.full[st], kb * 64, c1, c2, c3);
                    ++issued;
                }
            }
            // nothing of this block may be in flight when it ends, and the ring is about to be reused:
            // the last MMAs must have released their stages; after a failed wait, the loads already
            // issued must still land
            for (uint32_t g = issued > kStages ? issued - kStages : 0; g < issued; ++g) {
                const int st = g % kStages;
                if (!mbar_wait(&bar.empty[st], (g / kStages) & 1, &abort_s)) {
                    volatile int never = 0;
                    mbar_wait(&bar.full[st], (g / kStages) & 1, &never);
                }
            }
            if (qs.loads > 0) {
                volatile int never = 0;
                mbar_wait(&bar.qfull, (qs.loads - 1) & 1u, &never);
            }
        }
        __syncwarp();
        // the tail of the gather: the idle tile ring becomes copy slots
        if (gathers) {
            uint32_t phase = 0;
            int n_tail = kStages * stage_bytes / kCopySlotBytes;
            if (n_tail > kTailSlotsMax) n_tail = kTailSlotsMax;
            if (!abort_s) copy_units(a, k_stage0, bar.tail, n_tail, phase, &abort_s, lane);
            copiers_done(a, lane);
        }
    } else if (warp == 1) {
        // ================================================================== MMA issue
        if (lane == 0) {
            uint32_t it = 0;
            QState qs = {-1, 0, 0};
            Cursor cur;
            cursor_init(cur);
            Entry e;
            const uint64_t q_desc0 = umma_desc_sw128(smem_u32(q_img0));
            const uint64_t k_desc0 = umma_desc_sw128(smem_u32(k_stage0));
            const uint32_t stage_step = (uint32_t)stage_bytes >> 4;
            bool ok = true;
            while (ok && next_entry(a, cur, e)) {
                if (e.n_tiles == 0) continue;
                if (qs.unit != e.unit) {
                    if (qs.unit != -1) {
                        umma_commit(&bar.qfree);          // arrives once every MMA issued so far has completed
                        ++qs.frees;
                    }
                    ok = mbar_wait(&bar.qfull, qs.loads & 1u, &abort_s);
                    ++qs.loads;
                    qs.unit = e.unit;
                    if (!ok) break;
                    tc_fence_after_sync();
                }
                const bool sweep2 = e.phase != 0;
                const uint32_t idesc = sweep2 ? umma_idesc_bf16(128, a.r16) : umma_idesc_bf16(128, kTile);
                for (int t = 0; t < e.n_tiles; ++t) {
                    const uint32_t g = it + t;
                    const int st = g % kStages;
                    if (!mbar_wait(&bar.full[st], (g / kStages) & 1, &abort_s)) {
                        ok = false;
                        break;
                    }
                    const int buf = g % kBufs;
                    if (g >= kBufs && !mbar_wait(&bar.tempty[buf], ((g / kBufs) - 1) & 1, &abort_s)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint64_t k_desc = k_desc0 + (uint64_t)(st * stage_step);
                    const uint32_t d_tmem = tmem_base + buf * 128;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        if (ks < ksteps) {
                            const uint32_t qo = (uint32_t)((ks >> 2) * kQRegion + (ks & 3) * 32) >> 4;
                            const uint32_t ko = (uint32_t)((ks >> 2) * kRegion + (ks & 3) * 32) >> 4;
                            if (sweep2) umma_bf16(d_tmem, k_desc + ko, q_desc0 + qo, idesc, ks > 0);
                            else umma_bf16(d_tmem, q_desc0 + qo, k_desc + ko, idesc, ks > 0);
                        }
                    }
                    umma_commit(&bar.tfull[buf]);
                    umma_commit(&bar.empty[st]);
                }
                it += e.n_tiles;
            }
        }
        __syncwarp();
    } else if (warp < 2 + kComputeWarps) {
        // ================================================================== compute warps
        const int grp = (warp - 2) >> 2, quarter = warp & 3;
        const int L = quarter * 32 + lane;                 // tensor-memory lane of this thread
        const int tl = (int)threadIdx.x - 64;              // index among the compute threads
        const uint32_t taddr_grp = tmem_base + ((uint32_t)(quarter * 32) << 16) + grp * 128;
        const int Rp = a.Rp;
        uint32_t it = 0;
        Cursor cur;
        cursor_init(cur);
        Entry e;
        int aborted = 0;
        while (!aborted && next_entry(a, cur, e)) {
            if (e.phase == 0) {
                // ---------------------------------------------------------- statistics sweep (Eq. 1)
                unsigned long long *out = a.pstats + ((size_t)e.unit * a.n_stat_chunks + e.chunk) * 128;
                if (e.n_tiles == 0) continue;        // a chunk without keys: nobody reads its entries
                {
                    const int col0 = (L / Rp) * Rp;                 // warp-uniform: Rp is a multiple of 32
                    const int nslot = Rp >> 5;                      // 32-column slots this thread reduces
                    float m0 = -INFINITY, l0 = 0.f;
                    const int row = L % Rp;
                    const int limit0 = row < s.R ? min(e.n_r + row % s.alpha, e.j_end - 1) : -1;
                    const uint32_t taddr = taddr_grp + col0;
                    for (uint32_t g = it; g < it + e.n_tiles; ++g) {
                        if ((int)(g % kBufs) != grp) continue;
                        const int t = (int)(g - it);
                        if (!warp_wait(&bar.tfull[grp], (g / kBufs) & 1, &abort_s, lane)) break;
                        tc_fence_after_sync();
                        const int tile0 = e.j_begin + t * kTile;
                        const int j0 = tile0 + col0;
                        const bool fast = (tile0 + kTile - 1 <= e.n_r) && (tile0 + kTile - 1 < e.j_end);
                        for (int sl = 0; sl < nslot; ++sl) {
                            float x[32];
                            tmem_ld32(taddr + sl * 32, x);
                            if (sl + 1 == nslot) warp_release(&bar.tempty[grp], lane);
                            stats_update(x, fast, j0 + sl * 32, limit0, c, m0, l0);
                        }
                    }
                    part[grp][L] = make_float2(m0, l0);
                }
                it += e.n_tiles;
                compute_sync();
                // combine the compute groups and the column slices of each row, in a fixed order
                const int copies = 128 / Rp;
                if (tl < s.R) {
                    const int r = tl;
                    float M = -INFINITY;
                    for (int g = 0; g < kBufs; ++g)
                        for (int cp = 0; cp < copies; ++cp) M = fmaxf(M, part[g][r + cp * Rp].x);
                    float sum = 0.f;
                    for (int g = 0; g < kBufs; ++g)
                        for (int cp = 0; cp < copies; ++cp) {
                            const float2 p = part[g][r + cp * Rp];
                            if (p.y > 0.f) sum += p.y * fast_exp2((p.x - M) * c);
                        }
                    // published as it is written: no fence, no counter
                    st_relaxed_gpu_u64(out + r, stat_pack(M * c, sum));
                }
                // uniform over the compute warps: nobody leaves the list while others still synchronise
                int any;
                asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.s32 q, %1, 0;\n\t"
                             "bar.red.or.pred p, %2, %3, q;\n\tselp.s32 %0, 1, 0, p;\n\t}"
                             : "=r"(any) : "r"((int)abort_s), "n"(kBarCompute), "n"(kComputeThreads) : "memory");
                aborted = any;
                continue;
            }
            // -------------------------------------------------------------- scoring sweep (Eq. 2-4) + selection
            const int kw = num_windows(e.n, s.alpha, s.omega);
            const int budget = a.window_idx ? (s.budgets ? __ldg(s.budgets + e.b) : s.budget) : 0;
            int *unit_words = a.sync + kSyncTickets + kSyncWordsPerUnit * e.unit;
            if (e.n_tiles == 0) {
                // a unit without review context still gets its (empty) selection, from its first item
                if (a.window_idx && e.n_r <= 0 && e.chunk == 0) {
                    select_topk_block<kComputeThreads, kBarCompute, 64>(
                        topk_sm, a.window_scores + (size_t)e.unit * s.kw_max, 0, 0, s.k_max,
                        a.window_idx + (size_t)e.unit * s.k_max, a.kept_len + e.unit, e.n, s.alpha, s.omega);
                    compute_sync();
                    if (gathers && tl == 0) {
                        __threadfence();
                        st_release_gpu(unit_words + 2, 1);
                    }
                }
                continue;
            }
            // Eq. 1's normaliser of every row
            if (a.lse_obs) {
                if (tl < 128) {
                    float v = -INFINITY;
                    if (tl < s.R) {
                        const int g = tl / s.alpha, i = tl - g * s.alpha;
                        v = -1.4426950408889634f *
                            __ldg(a.lse_obs + ((size_t)e.b * s.hq + (size_t)e.h * s.G + g) * s.alpha + i);
                    }
                    neg_lse2[tl] = v;
                }
            } else {
                // merge the partial statistics of the unit's chunks: four threads share a row (each takes
                // every fourth chunk), then one of them merges their results; both in a fixed order
                constexpr int kMergers = kComputeThreads / 128;
                float2 *merged = &part[0][0];
                const int len1 = tc_chunk_len(e.n, cpu, 1);
                const int used1 = (e.n + len1 - 1) / len1;   // chunks of the unit that hold keys in the statistics sweep
                {
                    const int r = tl % 128, mp = tl / 128;
                    float M = -INFINITY, sum = 0.f;
                    const int used = r < s.R ? used1 : 0;
                    const unsigned long long *st = a.pstats + (size_t)e.unit * a.n_stat_chunks * 128 + r;
                    for (int c0 = mp; c0 < used; c0 += 8 * kMergers) {
                        float2 p[8];
                        // entries that have not been written yet read as zero: look again (bounded)
                        unsigned long long t0 = 0;
                        for (uint32_t spin = 1;; ++spin) {
                            bool all = true;
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const int cidx = c0 + u * kMergers;
                                p[u] = make_float2(-INFINITY, 0.f);
                                if (cidx < used) all &= stat_unpack(ld_relaxed_gpu_u64(st + (size_t)cidx * 128), p[u]);
                            }
                            if (all) break;
                            if (*static_cast<volatile int *>(&abort_s)) break;
                            __nanosleep(100);     // 512 threads look again: leave the L2 to the blocks still publishing
                            if ((spin & 63u) == 0u) {
                                const unsigned long long now = global_timer_ns();
                                if (t0 == 0) t0 = now;
                                else if (now - t0 > 2 * kWaitLimitNs) {
                                    abort_s = 1;
                                    break;
                                }
                            }
                        }
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
                    merged[mp * 128 + r] = make_float2(M, sum);
                }
                compute_sync();
                if (tl < 128) {
                    float v = -INFINITY;
                    if (tl < s.R) {
                        float M = -INFINITY, sum = 0.f;
#pragma unroll
                        for (int mp = 0; mp < kMergers; ++mp) {
                            const float2 p = merged[mp * 128 + tl];
                            if (p.y > 0.f) {
                                const float Mn = fmaxf(M, p.x);
                                sum = sum * fast_exp2(M - Mn) + p.y * fast_exp2(p.x - Mn);
                                M = Mn;
                            }
                        }
                        if (sum > 0.f) v = -(M + log2f(sum));
                    }
                    neg_lse2[tl] = v;
                }
            }
            compute_sync();
            {
                // token score of key L of every tile of the item -> t_chunk (and token_scores)
                const int n32 = a.r16 >> 5;
                const bool tail = (a.r16 & 16) != 0;
                for (uint32_t g = it; g < it + e.n_tiles; ++g) {
                    if ((int)(g % kBufs) != grp) continue;
                    const int t = (int)(g - it);
                    if (!warp_wait(&bar.tfull[grp], (g / kBufs) & 1, &abort_s, lane)) break;
                    tc_fence_after_sync();
                    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
                    for (int sl = 0; sl < n32; ++sl) {
                        float v[32];
                        tmem_ld32(taddr_grp + sl * 32, v);
                        if (sl + 1 == n32 && !tail) warp_release(&bar.tempty[grp], lane);
                        score_accumulate<32>(v, neg_lse2 + sl * 32, c, a0, a1, a2, a3);
                    }
                    if (tail) {
                        float vt[16];
                        tmem_ld16(taddr_grp + n32 * 32, vt);
                        warp_release(&bar.tempty[grp], lane);
                        score_accumulate<16>(vt, neg_lse2 + n32 * 32, c, a0, a1, a2, a3);
                    }
                    const float tj = (a0 + a1) + (a2 + a3);
                    const int j = e.j_begin + t * kTile + L;
                    if (j < e.j_end) {
                        t_chunk[j - e.j_begin] = tj;
                        if (a.token_scores) a.token_scores[(size_t)e.unit * s.nr_max + j] = tj;
                    }
                }
            }
            it += e.n_tiles;
            compute_sync();
            // Eq. 3-4: the item's windows (its first key is a multiple of omega)
            {
                const int n_tok = e.j_end - e.j_begin;
                float *ws_out = a.window_scores + (size_t)e.unit * s.kw_max + e.j_begin / s.omega;
                const int n_win = (n_tok + s.omega - 1) / s.omega;
                if (s.omega == 16 || s.omega == 8 || s.omega == 32 || s.omega == 4) {
                    // consecutive windows go to different warps so that all four schedulers take part
                    for (int i = tl; i < n_win; i += kComputeThreads) {
                        const int lo = i * s.omega, size = min(s.omega, n_tok - lo);
                        float r;
                        if (s.omega == 16) r = pool_window_sorted<16>(t_chunk + lo, size, s.p);
                        else if (s.omega == 8) r = pool_window_sorted<8>(t_chunk + lo, size, s.p);
                        else if (s.omega == 32) r = pool_window_sorted<32>(t_chunk + lo, size, s.p);
                        else r = pool_window_sorted<4>(t_chunk + lo, size, s.p);
                        ws_out[i] = r;
                    }
                } else if (s.omega == 64 || s.omega == 128) {
                    // one warp per window
                    for (int lw = tl >> 5; lw < n_win; lw += kComputeWarps) {
                        const int lo = lw * s.omega, size = min(s.omega, n_tok - lo);
                        const float r = s.omega == 64 ? pool_window_warp<64>(t_chunk + lo, size, s.p, lane)
                                                      : pool_window_warp<128>(t_chunk + lo, size, s.p, lane);
                        if (lane == 0) ws_out[lw] = r;
                    }
                } else {
                    for (int lw = tl; lw < n_win; lw += kComputeThreads) {
                        const int lo = lw * s.omega;
                        ws_out[lw] = pool_top_p(t_chunk + lo, min(s.omega, n_tok - lo), s.p);
                    }
                }
            }
            const int len2 = tc_chunk_len(e.n_r, cpu, s.omega);
            const int used2 = (e.n_r + len2 - 1) / len2;   // chunks of the unit that hold keys in this sweep
            // The block of the unit's last chunk selects for the unit (and clears the unit's words); the
            // other blocks only count themselves, without waiting for an answer.
            int any;
            asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.s32 q, %1, 0;\n\t"
                         "bar.red.or.pred p, %2, %3, q;\n\tselp.s32 %0, 1, 0, p;\n\t}"
                         : "=r"(any) : "r"((int)abort_s), "n"(kBarCompute), "n"(kComputeThreads) : "memory");
            aborted = any;
            if (aborted) break;
            if (e.chunk != used2 - 1) {
                // release, cumulative: publishes the window scores the compute warps wrote before the barrier
                if (tl == 0) red_release_gpu_add(unit_words, 1);
            } else {
                if (tl == 0 && poll_until_at_least(unit_words, used2 - 1, &abort_s)) {
                    atomicExch(unit_words, 0);       // every other block of the unit has read what it needs
                    atomicExch(unit_words + 1, 0);
                }
                asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.s32 q, %1, 0;\n\t"
                             "bar.red.or.pred p, %2, %3, q;\n\tselp.s32 %0, 1, 0, p;\n\t}"
                             : "=r"(any) : "r"((int)abort_s), "n"(kBarCompute), "n"(kComputeThreads) : "memory");
                aborted = any;
                if (aborted) break;
                if (!a.lse_obs) {
                    // the unit's statistics entries go back to "not written" for the next launch
                    const int len1 = tc_chunk_len(e.n, cpu, 1);
                    const int used1 = (e.n + len1 - 1) / len1;
                    unsigned long long *st = a.pstats + (size_t)e.unit * a.n_stat_chunks * 128;
                    for (int i = tl; i < used1 * 128; i += kComputeThreads) st[i] = 0ull;
                }
                if (a.window_idx) {
                    select_topk_block<kComputeThreads, kBarCompute, 64>(
                        topk_sm, a.window_scores + (size_t)e.unit * s.kw_max, kw,
                        num_selected_capped(e.n, s.alpha, s.omega, budget, s.k_max), s.k_max,
                        a.window_idx + (size_t)e.unit * s.k_max, a.kept_len + e.unit, e.n, s.alpha, s.omega);
                    if (gathers) {
                        // publish: the indices every compute thread wrote, then the flag the copy warps poll
                        __threadfence();
                        compute_sync();
                        if (tl == 0) st_release_gpu(unit_words + 2, 1);
                    }
                }
            }
            compute_sync();   // t_chunk, neg_lse2 and the selection scratch are reused by the next item
        }
    } else {
        // ================================================================== copy warps
        if (gathers) {
            const int cw = warp - (2 + kComputeWarps);
            uint32_t phase = 0;
            copy_units(a, copy_ring + (size_t)cw * kCopySlots * kCopySlotBytes, bar.copy[cw], kCopySlots, phase, &abort_s,
                       lane);
            copiers_done(a, lane);
        }
    }

    // ------------------------------------------------------------------ teardown
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (threadIdx.x == 0 && abort_s) atomicOr(a.status, kStatusWaitExpired);
    if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn pipe_encode_fn()
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

// Tensor map of a bf16 tensor with the head dimension innermost: dimension 0 is the head dimension;
// `dims` (size, stride in bytes, box) follow in the given order, except that dimensions of size one,
// which carry no address information, get a stride that keeps the map valid.  128-byte swizzle.
struct MapDim {
    unsigned long long size, stride;
    unsigned box;
};
bool encode_map(const void *base, int head_dim, const MapDim dims[3], CUtensorMap *tmap, const char *what)
{
    EncodeTiledFn enc = pipe_encode_fn();
    if (!enc) {
        set_error_detail("cuTensorMapEncodeTiled is not available from the driver");
        return false;
    }
    unsigned long long running = (unsigned long long)head_dim * 2ull;
    cuuint64_t gdim[4] = {(cuuint64_t)head_dim, 0, 0, 0}, gstride[3];
    cuuint32_t box[4] = {64, 1, 1, 1}, estr[4] = {1, 1, 1, 1};
    for (int i = 0; i < 3; ++i) {
        unsigned long long stride = dims[i].size == 1 ? running : dims[i].stride;
        if (stride == 0 || stride % 16 || stride >= (1ull << 40) || dims[i].size > 0xffffffffull || dims[i].box > 256) {
            set_error_detail("%s layout cannot be described by a tensor map (dimension %d: size %llu, stride %llu bytes)",
                             what, i, dims[i].size, stride);
            return false;
        }
        gdim[i + 1] = dims[i].size;
        gstride[i] = stride;
        box[i + 1] = dims[i].box;
        const unsigned long long span = stride * dims[i].size;
        if (span > running) running = span;
    }
    const CUresult r = enc(tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), gdim, gstride, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error_detail("cuTensorMapEncodeTiled (%s) failed with code %d", what, (int)r);
        return false;
    }
    return true;
}

struct PipeDevice {
    bool known = false;
    int cc_major = -1, sm_count = 0, cooperative = 0;
    int blocks_per_sm = -1;
};
std::mutex g_pipe_mutex;
PipeDevice g_pipe_device[kMaxDevices];

PipeDevice *pipe_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return nullptr;
    }
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    PipeDevice &info = g_pipe_device[dev];
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

size_t pipe_smem_bytes(int kblocks)
{
    return 1024 + (size_t)kblocks * kQRegion + (size_t)kStages * kblocks * kRegion +
           (size_t)kCopyWarps * kCopySlots * kCopySlotBytes;
}

}  // namespace

bool group_pipeline_supported(const KShape &ks, int dtype)
{
    const PipeDevice *di = pipe_device();
    // the Q image is fetched as one box of alpha positions x G heads: positions must be the faster dimension
    const bool q_order = (ks.alpha == 1 || ks.G == 1 || ks.qst <= ks.qsh);
    return di && dtype == WKV_BF16 && (ks.d == 64 || ks.d == 128) && ks.R <= 128 && ks.alpha <= 128 && ks.G <= 128 &&
           ks.omega <= kTcMaxWindow && q_order && di->cc_major == 10 && di->cooperative && di->sm_count > 0;
}

bool group_pipeline_can_gather(const KShape &ks, int elem_bytes, int n_tensors)
{
    const long long row_bytes = (long long)ks.d * elem_bytes;
    return n_tensors > 0 && n_tensors <= 2 * WKV_MAX_GROUP_LAYERS && row_bytes <= kCopySlotBytes && row_bytes % 16 == 0;
}

int launch_group_pipeline(const KShape &ks, const void *q, const void *k, float *window_scores, float *token_scores,
                          int *window_idx, int *kept_len, void *workspace, const Workspace &ws, cudaStream_t stream,
                          const float *lse_obs, const PipeGather *gather)
{
    PipeDevice *di = pipe_device();
    if (!di) {
        set_error_detail("no current CUDA device, or its ordinal is beyond %d", kMaxDevices - 1);
        return WKV_ERR_CUDA;
    }
    alignas(64) CUtensorMap kmap, qmap;
    // keys: token, head and batch in order of increasing stride (dimensions of size one last)
    int slot[3] = {1, 2, 3};
    {
        struct D {
            MapDim m;
            int which;
        } d3[3] = {
            {{(unsigned long long)(ks.cu ? ks.total_rows : ks.max_seqlen), (unsigned long long)ks.st * 2ull, (unsigned)kTile}, 0},
            {{(unsigned long long)ks.hkv, (unsigned long long)ks.sh * 2ull, 1u}, 1},
            {{(unsigned long long)(ks.cu ? 1 : ks.batch), (unsigned long long)ks.sb * 2ull, 1u}, 2},
        };
        std::stable_sort(d3, d3 + 3, [](const D &x, const D &y) {
            const bool x1 = x.m.size == 1, y1 = y.m.size == 1;
            if (x1 != y1) return y1;
            return !x1 && x.m.stride < y.m.stride;
        });
        MapDim dims[3];
        for (int i = 0; i < 3; ++i) {
            dims[i] = d3[i].m;
            slot[d3[i].which] = i + 1;
        }
        if (!encode_map(k, ks.d, dims, &kmap, "key")) return WKV_ERR_UNSUPPORTED;
    }
    {
        // queries: (position in the observation window, query head, sequence); one box = one unit's rows
        const MapDim dims[3] = {
            {(unsigned long long)ks.alpha, (unsigned long long)ks.qst * 2ull, (unsigned)ks.alpha},
            {(unsigned long long)ks.hq, (unsigned long long)ks.qsh * 2ull, (unsigned)ks.G},
            {(unsigned long long)ks.batch, (unsigned long long)ks.qsb * 2ull, 1u},
        };
        if (!encode_map(q, ks.d, dims, &qmap, "query")) return WKV_ERR_UNSUPPORTED;
    }

    PipeArgs a;
    a.s = ks;
    a.pstats = reinterpret_cast<unsigned long long *>(static_cast<char *>(workspace) + ws.pstats_off);
    a.window_scores = window_scores;
    a.token_scores = token_scores;
    a.lse_obs = lse_obs;
    a.window_idx = window_idx;
    a.kept_len = kept_len;
    a.status = reinterpret_cast<int *>(static_cast<char *>(workspace) + ws.status_off);
    a.sync = reinterpret_cast<int *>(static_cast<char *>(workspace) + ws.sync_off);
    a.n_stat_chunks = ws.n_stat_chunks;
    const int units = ks.batch * ks.hkv;
    const PipePlan plan = pipe_plan(units, ks.max_seqlen, ks.d);
    a.chunks_per_unit = plan.chunks_per_unit;
    a.units_per_wave = plan.units_per_wave;
    a.n_waves = (units + plan.units_per_wave - 1) / plan.units_per_wave;
    a.skew = (plan.skew && !lse_obs) ? 1 : 0;
    a.kblocks = ks.d / 64;
    a.slot_tok = slot[0];
    a.slot_h = slot[1];
    a.slot_b = slot[2];
    a.r16 = (ks.R + 15) / 16 * 16;
    a.Rp = ks.R <= 32 ? 32 : (ks.R <= 64 ? 64 : 128);
    a.q_copies = 128 / a.Rp;
    a.n_tensors = 0;
    a.keep_capacity = 0;
    a.cu_out = nullptr;
    a.row_bytes = ks.d * 2;
    a.src_row_stride = ks.st * 2;
    a.obs_slots = (ks.alpha + ks.omega - 1) / ks.omega;
    a.rows_per_job = std::max(1, std::min(ks.omega, kCopySlotBytes / a.row_bytes));
    a.subs_per_window = (ks.omega + a.rows_per_job - 1) / a.rows_per_job;
    if (gather && window_idx) {
        a.n_tensors = gather->n_tensors;
        a.keep_capacity = gather->keep_capacity;
        a.cu_out = gather->cu_out;
        a.tab = *gather->tab;
    }

    const size_t smem = pipe_smem_bytes(a.kblocks);
    const void *fn = reinterpret_cast<const void *>(group_pipeline_tc);
    cudaError_t err = cudaSuccess;
    {
        std::lock_guard<std::mutex> lock(g_pipe_mutex);
        if (di->blocks_per_sm < 0) {
            const size_t smem_max = pipe_smem_bytes(2);
            err = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
            if (err == cudaSuccess)
                err = cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
            int occ = 0;
            if (err == cudaSuccess) err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, fn, kThreads, smem_max);
            if (err == cudaSuccess) {
                if (occ < 1) {
                    cudaFuncAttributes fa;
                    (void)cudaFuncGetAttributes(&fa, fn);
                    set_error_detail("pipelined group kernel does not fit an SM (%d threads, %d registers, %zu + %zu bytes "
                                     "of shared memory)", kThreads, fa.numRegs, smem_max, fa.sharedSizeBytes);
                    return WKV_ERR_CUDA;
                }
                di->blocks_per_sm = occ;
            }
        }
    }
    // persistent blocks, one per SM at most; every block of a cooperative launch is resident, which the
    // hand-overs between blocks rely on
    int grid = plan.units_per_wave * plan.chunks_per_unit;
    if (grid > di->sm_count) grid = di->sm_count;
    if (err == cudaSuccess) {
        void *params[3] = {&kmap, &qmap, &a};
        err = cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kThreads), params, smem, stream);
    }
    if (err != cudaSuccess) {
        set_error_detail("pipelined group kernel (grid %d x %d threads, %zu bytes of shared memory): %s", grid, kThreads,
                         smem, cudaGetErrorString(err));
        return WKV_ERR_CUDA;
    }
    count_launches(1);
    return WKV_OK;
}

}  // namespace wkv
