// Measurement aid (no counterpart in the paper): the rate at which this GPU evaluates
// ex2.approx.ftz.f32, the instruction both sweeps of the score kernels spend most of their issue
// slots on.  The benchmark times this kernel with CUDA events and uses the measured rate, instead of
// an assumed one, as the special-function floor of the score stage.
#include "tc_common.cuh"
#include "wkv_internal.cuh"

namespace wkv {
namespace {

constexpr int kChains = 8;   // independent dependency chains per thread

__global__ void __launch_bounds__(1024)
ex2_rate_kernel(float *out, int iters, float seed)
{
    float x[kChains];
#pragma unroll
    for (int i = 0; i < kChains; ++i) x[i] = seed + 0.001f * (float)(threadIdx.x + i);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < kChains; ++i) x[i] = tc::fast_exp2(x[i]);   // 2^x of a value in [-0.5, 1] lies in [0.7, 2]
#pragma unroll
        for (int i = 0; i < kChains; ++i) x[i] -= 1.0f;                  // minus one: back in [-0.3, 1]; one FADD per ex2
    }
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < kChains; ++i) acc += x[i];
    if (acc == 123.456f) out[0] = acc;    // never true in practice; keeps the chains alive
}

// Column sums across the lanes of a warp: every lane holds 32 values (a 32 x 32 block, one row per
// lane), and after 31 shuffle-and-add steps (halving exchange: 16 + 8 + 4 + 2 + 1) lane l holds the sum
// of column l over the 32 lanes.  This is the cross-lane reduction a single-sweep score kernel would
// need once per tile element (whichever operand sits on the tensor-memory lanes, either the row
// normaliser of Eq. 1 or the column sum of Eq. 2 runs across lanes); its rate, set beside the ex2
// rate, says whether dropping the second sweep's exponentials could pay for it.
__global__ void __launch_bounds__(1024)
colsum_rate_kernel(float *out, int iters, float seed)
{
    const int lane = threadIdx.x & 31;
    float v[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = seed + 0.001f * (float)(threadIdx.x + i);
    float keep = 0.f;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
            const bool upper = (lane & o) != 0;
#pragma unroll
            for (int i = 0; i < o; ++i) {
                const float send = upper ? v[i] : v[i + o];
                const float recv = __shfl_xor_sync(0xffffffffu, send, o);
                v[i] = (upper ? v[i + o] : v[i]) + recv;
            }
        }
        keep += v[0];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = v[0] * 0.03125f + 0.001f * (float)i;   // next block of values
    }
    if (keep == 123.456f) out[0] = keep;
}

}  // namespace
}  // namespace wkv

extern "C" int wkv_probe_colsum_rate(float *scratch_dev, int32_t blocks, int32_t threads, int32_t iters,
                                     int64_t *elements_per_launch, void *cuda_stream)
{
    using namespace wkv;
    if (!scratch_dev) {
        set_error_detail("scratch_dev is NULL");
        return WKV_ERR_NULL;
    }
    if (blocks < 1 || threads < 32 || threads > 1024 || threads % 32 || iters < 1) {
        set_error_detail("probe shape: blocks %d, threads %d, iters %d", blocks, threads, iters);
        return WKV_ERR_SHAPE;
    }
    colsum_rate_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(scratch_dev, iters, 0.25f);
    if (elements_per_launch) *elements_per_launch = (int64_t)blocks * threads * 32 * iters;
    count_launches(1);
    return check_cuda(cudaGetLastError(), "column-sum probe kernel");
}

extern "C" int wkv_probe_ex2_rate(float *scratch_dev, int32_t blocks, int32_t threads, int32_t iters,
                                  int64_t *ex2_per_launch, void *cuda_stream)
{
    using namespace wkv;
    if (!scratch_dev) {
        set_error_detail("scratch_dev is NULL");
        return WKV_ERR_NULL;
    }
    if (blocks < 1 || threads < 32 || threads > 1024 || threads % 32 || iters < 1) {
        set_error_detail("probe shape: blocks %d, threads %d, iters %d", blocks, threads, iters);
        return WKV_ERR_SHAPE;
    }
    ex2_rate_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(scratch_dev, iters, 0.25f);
    if (ex2_per_launch) *ex2_per_launch = (int64_t)blocks * threads * kChains * iters;
    count_launches(1);
    return check_cuda(cudaGetLastError(), "ex2 probe kernel");
}
