// Stand-alone budgeted window selection (sentence after Eq. 4): one thread block per unit.
#include "topk_block.cuh"

namespace wkv {
namespace {

constexpr int kThreads = 1024;

__global__ void __launch_bounds__(kThreads)
select_topk_kernel(KShape s, const float *__restrict__ window_scores, int *__restrict__ window_idx,
                   int *__restrict__ kept_len)
{
    __shared__ TopkSmem sm;
    const int unit = blockIdx.x;
    const int b = unit / s.hkv;
    const SeqInfo si = seq_info(s, b);
    const int kw = num_windows(si.n, s.alpha, s.omega);
    const int k = num_selected_capped(si.n, s.alpha, s.omega, si.budget, s.k_max);
    select_topk_block<kThreads>(sm, window_scores + (size_t)unit * s.kw_max, kw, k, s.k_max,
                                window_idx + (size_t)unit * s.k_max, kept_len + unit, si.n, s.alpha, s.omega);
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
