// A layer group as a replayable object.  An engine that keeps its K/V pools and compact caches at
// fixed addresses calls the same group with the same arguments for every request; recording the
// launches of that call once in a CUDA graph and replaying the graph removes most of the gap at the
// kernel boundary that two separate launches on a stream leave.  The plan holds nothing but the graph: inputs, outputs and the
// workspace stay the caller's, and what a launch computes is exactly what wkv_compress_group
// computes on the buffers' contents at that moment.
#include "wkv_internal.cuh"

#include <new>

struct wkv_group_plan {
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    uint64_t kernels = 0;   // kernel launches one replay stands for
};

using namespace wkv;

extern "C" {

int wkv_group_plan_create(const wkv_shape *s, int32_t n_layers, const void *q_obs_leader, const float *lse_obs,
                          const void *const *k_layers, const void *const *v_layers, void *const *k_out_layers,
                          void *const *v_out_layers, float *window_scores, int32_t *window_idx,
                          int32_t *kept_len, const int32_t *cu_seqlens_out, int32_t keep_capacity,
                          void *workspace, size_t workspace_bytes, wkv_group_plan **plan_out)
{
    if (!plan_out) {
        set_error_detail("plan_out is NULL");
        return WKV_ERR_NULL;
    }
    *plan_out = nullptr;
    cudaStream_t cap = nullptr;
    int st = check_cuda(cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking), "stream for recording the plan");
    if (st != WKV_OK) return st;
    wkv_group_plan *plan = new (std::nothrow) wkv_group_plan;
    if (!plan) {
        cudaStreamDestroy(cap);
        set_error_detail("out of host memory");
        return WKV_ERR_CUDA;
    }
    st = check_cuda(cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal), "begin recording the plan");
    if (st == WKV_OK) {
        const uint64_t before = launches_so_far();
        // the arguments are validated here exactly as by the direct call; nothing runs yet
        const int call = compress_group_entry(s, n_layers, q_obs_leader, lse_obs, k_layers, v_layers, k_out_layers,
                                              v_out_layers, window_scores, window_idx, kept_len, cu_seqlens_out,
                                              keep_capacity, workspace, workspace_bytes, cap);
        plan->kernels = launches_so_far() - before;
        const cudaError_t end = cudaStreamEndCapture(cap, &plan->graph);   // always ends the recording
        st = call != WKV_OK ? call : check_cuda(end, "end recording the plan");
        // what was counted while recording did not run
        count_launches(-(int)plan->kernels);
    }
    if (st == WKV_OK) st = check_cuda(cudaGraphInstantiate(&plan->exec, plan->graph, 0), "instantiating the plan");
    cudaStreamDestroy(cap);
    if (st != WKV_OK) {
        if (plan->exec) cudaGraphExecDestroy(plan->exec);
        if (plan->graph) cudaGraphDestroy(plan->graph);
        delete plan;
        return st;
    }
    *plan_out = plan;
    return WKV_OK;
}

int wkv_group_plan_launch(wkv_group_plan *plan, void *cuda_stream)
{
    if (!plan || !plan->exec) {
        set_error_detail("plan is NULL");
        return WKV_ERR_NULL;
    }
    const int st = check_cuda(cudaGraphLaunch(plan->exec, static_cast<cudaStream_t>(cuda_stream)), "launching the plan");
    if (st == WKV_OK) count_launches((int)plan->kernels);
    return st;
}

void wkv_group_plan_destroy(wkv_group_plan *plan)
{
    if (!plan) return;
    if (plan->exec) cudaGraphExecDestroy(plan->exec);
    if (plan->graph) cudaGraphDestroy(plan->graph);
    delete plan;
}

}  // extern "C"
