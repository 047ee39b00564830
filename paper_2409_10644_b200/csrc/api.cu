// Status reporting of libmcsd.
#include <atomic>

#include "common.cuh"

namespace mcsd {
static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = static_cast<int>(e); }
static std::atomic<long long> g_launches{0};
void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
}  // namespace mcsd

extern "C" const char* mcsd_status_string(int status) {
    switch (status) {
        case MCSD_OK: return "ok";
        case MCSD_ERR_NULL: return "a required pointer is NULL";
        case MCSD_ERR_BAD_SHAPE: return "a size or an alignment is out of the supported range";
        case MCSD_ERR_NOT_BFS: return "parent array is not a level-ordered forest";
        case MCSD_ERR_BAD_DTYPE: return "unsupported dtype for this shape";
        case MCSD_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case MCSD_ERR_CUDA: return "CUDA call failed";
        case MCSD_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case MCSD_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch of this entry point";
        default: return "unknown status";
    }
}

extern "C" int mcsd_last_cuda_error(void) { return mcsd::g_last_cuda_error; }

extern "C" long long mcsd_launch_count(void) { return mcsd::g_launches.load(std::memory_order_relaxed); }

extern "C" int mcsd_workspace_status(const void* workspace, void* stream) {
    if (workspace == nullptr) return MCSD_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t host[2] = {0, 0};
    MCSD_CUDA_CHECK(cudaMemcpyAsync(host, workspace, sizeof(host), cudaMemcpyDeviceToHost, s));
    MCSD_CUDA_CHECK(cudaStreamSynchronize(s));
    return host[0] == 0 ? MCSD_OK : MCSD_ERR_TIMEOUT;
}
