// Multi-candidate accept/reject from probability rows (Fig. 1 steps 4-6 of the paper): entry points.
// The kernels are in verify_kernels.cuh.
#include <mutex>

#include "verify_kernels.cuh"

extern "C" size_t mcsd_verify_tree_workspace_bytes(int B, int N, int V) {
    (void)V;
    if (B < 1 || N < 1) return 0;
    return mcsd::verify_tickets_offset(B, N) + mcsd::align_up(sizeof(int) * (size_t)B, 256);
}

extern "C" int mcsd_verify_tree(const float* p, const float* q, const int32_t* tokens, const int32_t* parent,
                                const int32_t* level_start, int n_levels, int n_roots, const int32_t* gamma,
                                const float* u_accept, const float* u_bonus, int B, int N, int V,
                                int32_t* accept_len, int32_t* out_tokens, int32_t* out_nodes, int32_t* best_root,
                                int32_t* next_roots, int R, void* workspace, size_t workspace_bytes, void* stream) {
    if (!p || !q || !tokens || !parent || !level_start || !u_accept || !u_bonus || !accept_len || !out_tokens ||
        !out_nodes || !best_root || !workspace)
        return MCSD_ERR_NULL;
    if (B < 1 || N < 1 || V < 1 || N > MCSD_MAX_NODES || B > 65535) return MCSD_ERR_BAD_SHAPE;
    if (n_levels < 1 || n_levels > N || n_roots < 1 || n_roots > N) return MCSD_ERR_BAD_SHAPE;
    if (R < 0 || R > 32) return MCSD_ERR_BAD_SHAPE;
    if (R > 0 && !next_roots) return MCSD_ERR_NULL;
    if (workspace_bytes < mcsd_verify_tree_workspace_bytes(B, N, V)) return MCSD_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    auto* state = reinterpret_cast<mcsd::NodeState*>(static_cast<char*>(workspace) + sizeof(mcsd::WorkspaceHeader));
    const mcsd::ProbRows rows{p, q};
    int* tickets = reinterpret_cast<int*>(static_cast<char*>(workspace) + mcsd::verify_tickets_offset(B, N));
    mcsd::verify_tree_kernel<mcsd::ProbRows><<<dim3(N, B), mcsd::kVerifyThreads, 0, s>>>(
        rows, tokens, parent, level_start, n_levels, n_roots, gamma, u_accept, u_bonus, N, V, state, tickets, accept_len,
        out_tokens, out_nodes, best_root, R > 0 ? next_roots : nullptr, R);
    MCSD_CUDA_CHECK(cudaGetLastError());
    mcsd::count_launches(1);
    return MCSD_OK;
}

extern "C" int mcsd_sample_roots(const float* p, const float* q, const int32_t* accept_len, const int32_t* out_nodes,
                                 const int32_t* best_root, int n_levels, const float* u_roots, int B, int N, int V,
                                 int R, int32_t* next_roots, const void* workspace, size_t workspace_bytes,
                                 void* stream) {
    if (!p || !q || !accept_len || !out_nodes || !best_root || !u_roots || !next_roots || !workspace) return MCSD_ERR_NULL;
    if (B < 1 || N < 1 || V < 1 || N > MCSD_MAX_NODES || B > 65535) return MCSD_ERR_BAD_SHAPE;
    if (n_levels < 1 || n_levels > N || R < 1 || R > 32) return MCSD_ERR_BAD_SHAPE;
    if (workspace_bytes < mcsd_verify_tree_workspace_bytes(B, N, V)) return MCSD_ERR_WORKSPACE_TOO_SMALL;
    const auto* state = reinterpret_cast<const mcsd::NodeState*>(static_cast<const char*>(workspace) +
                                                                sizeof(mcsd::WorkspaceHeader));
    const mcsd::ProbRows rows{p, q};
    mcsd::sample_roots_kernel<mcsd::ProbRows><<<B, mcsd::kVerifyThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        rows, state, accept_len, out_nodes, best_root, n_levels, u_roots, N, V, R, next_roots);
    MCSD_CUDA_CHECK(cudaGetLastError());
    mcsd::count_launches(1);
    return MCSD_OK;
}

// ------------------------------------------------------------------------------------------------------
// Variant with built-in scratch, for callers that cannot allocate device memory.
// ------------------------------------------------------------------------------------------------------
namespace mcsd {

// Scratch that lives in the library image itself: one copy per GPU that loads the library, held until the
// process exits.  Layout as a workspace of the largest problem: header, MCSD_STATIC_VERIFY_MAX_STATES node states, one
// ticket per sequence (at most as many sequences as states).
constexpr size_t kStaticScratchBytes = sizeof(WorkspaceHeader) + sizeof(NodeState) * (size_t)MCSD_STATIC_VERIFY_MAX_STATES +
                                       256 + sizeof(int) * (size_t)MCSD_STATIC_VERIFY_MAX_STATES + 256;
static __device__ __align__(256) unsigned char g_static_verify_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static std::mutex g_static_mutex;
static void* g_static_ptr[kMaxDevices] = {};

// In host code the array's name is only a handle; the address kernels can use has to be asked for, once
// per device, with that device current.
static int static_scratch_for_current_device(void** out) {
    int dev = -1;
    MCSD_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return MCSD_ERR_BAD_SHAPE;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (g_static_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        MCSD_CUDA_CHECK(cudaGetSymbolAddress(&ptr, g_static_verify_scratch));
        if (ptr == nullptr) return MCSD_ERR_CUDA;
        g_static_ptr[dev] = ptr;
    }
    *out = g_static_ptr[dev];
    return MCSD_OK;
}

}  // namespace mcsd

extern "C" int mcsd_verify_tree_static(const float* p, const float* q, const int32_t* tokens, const int32_t* parent,
                                       const int32_t* level_start, int n_levels, int n_roots, const int32_t* gamma,
                                       const float* u_accept, const float* u_bonus, int B, int N, int V,
                                       int32_t* accept_len, int32_t* out_tokens, int32_t* out_nodes,
                                       int32_t* best_root, int32_t* next_roots, int R, void* stream) {
    if (B >= 1 && N >= 1 && (long long)B * N > MCSD_STATIC_VERIFY_MAX_STATES) return MCSD_ERR_STATIC_LIMIT;
    void* scratch = nullptr;
    const int st = mcsd::static_scratch_for_current_device(&scratch);
    if (st != MCSD_OK) return st;
    // the array keeps whatever the previous call left; the status line and this problem's tickets must start at zero
    MCSD_CUDA_CHECK(cudaMemsetAsync(scratch, 0, sizeof(mcsd::WorkspaceHeader), static_cast<cudaStream_t>(stream)));
    if (B >= 1 && N >= 1)
        MCSD_CUDA_CHECK(cudaMemsetAsync(static_cast<char*>(scratch) + mcsd::verify_tickets_offset(B, N), 0, sizeof(int) * (size_t)B,
                                        static_cast<cudaStream_t>(stream)));
    return mcsd_verify_tree(p, q, tokens, parent, level_start, n_levels, n_roots, gamma, u_accept, u_bonus, B, N, V,
                            accept_len, out_tokens, out_nodes, best_root, next_roots, R, scratch,
                            mcsd::kStaticScratchBytes, stream);
}
