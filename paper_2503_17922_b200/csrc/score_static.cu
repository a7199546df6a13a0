// wkv_score_windows_static: the scoring stage for callers that cannot provide scratch memory.
//
// Some hosts of this library run where device allocation is off the table: inside a serving
// engine that has handed every byte of HBM to its own KV-cache pool at start-up, in a callback
// that must not synchronise the device, or under a memory budget audited at load time.  Such a
// caller cannot size and allocate the workspace wkv_score_windows() asks for.  This entry point
// needs none: its partial row statistics live in a fixed array that is part of the library image.
// Every GPU that loads the library therefore holds WKV_STATIC_SCRATCH_BYTES of device memory
// until the process exits, whether or not the entry point is ever called.
#include "wkv_internal.cuh"

#include <mutex>

namespace wkv {
namespace {

// The one scratch area, shared by every call on a device.  In host code this name is only a
// handle for cudaGetSymbolAddress(); the device address is looked up once per device below.
static __device__ __align__(256) unsigned char g_static_scratch[WKV_STATIC_SCRATCH_BYTES];

std::mutex g_setup_mutex;
void *g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up on the first call per device).
int static_scratch(void **out)
{
    int dev = -1;
    int st = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
    if (st != WKV_OK) return st;
    if (dev < 0 || dev >= kMaxDevices) {
        set_error_detail("device ordinal %d outside 0..%d", dev, kMaxDevices - 1);
        return WKV_ERR_LIMIT;
    }
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        st = check_cuda(cudaGetSymbolAddress(&p, g_static_scratch), "cudaGetSymbolAddress(static scratch)");
        if (st != WKV_OK) return st;
        if (!p || (reinterpret_cast<uintptr_t>(p) & 255u)) {
            set_error_detail("static scratch has no usable device address");
            return WKV_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return WKV_OK;
}

}  // namespace
}  // namespace wkv

using namespace wkv;

extern "C" int wkv_score_windows_static(const wkv_shape *s, const void *q_obs, const void *k_leader,
                                        float *window_scores, float *token_scores, int32_t *device_status,
                                        void *cuda_stream)
{
    KShape ks;
    int st = resolve(s, ks);
    if (st != WKV_OK) return st;
    if (!q_obs || !k_leader || !window_scores) {
        set_error_detail("q_obs / k_leader / window_scores is NULL");
        return WKV_ERR_NULL;
    }
    const Workspace ws = plan_workspace(ks);
    // window_scores is the caller's here, so the part of the workspace that would hold them is not needed
    if (ws.scores_off > (size_t)WKV_STATIC_SCRATCH_BYTES) {
        set_error_detail("this shape needs %zu bytes of scratch, the built-in area holds %zu: "
                         "use wkv_score_windows with a caller-provided workspace",
                         ws.scores_off, (size_t)WKV_STATIC_SCRATCH_BYTES);
        return WKV_ERR_LIMIT;
    }
    void *scratch = nullptr;
    st = static_scratch(&scratch);
    if (st != WKV_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the status word and the grid-synchronisation words behind it are the only part of the area
    // that must start from zero; the kernels write every statistic they later read
    st = check_cuda(cudaMemsetAsync(static_cast<char *>(scratch) + ws.status_off, 0, ws.stats_off - ws.status_off,
                                    stream),
                    "clearing the status and synchronisation words");
    if (st != WKV_OK) return st;
    st = do_score(s, ks, ws, q_obs, k_leader, window_scores, token_scores, nullptr, nullptr, scratch, stream);
    if (st != WKV_OK) return st;
    if (device_status)
        st = check_cuda(cudaMemcpyAsync(device_status, static_cast<char *>(scratch) + ws.status_off, sizeof(int),
                                        cudaMemcpyDeviceToDevice, stream),
                        "copy of the status word");
    return st;
}
