// Topology-aware causal mask of a token tree as per-node ancestor bitsets (Section 2.2, Fig. 1 step 2;
// built once for the deepest tree so that the dynamic sliced mask of Section 3.2 is a prefix of its rows).
#include "common.cuh"

namespace mcsd {

struct TreeArg {
    int32_t parent[MCSD_MAX_NODES];
};

// One thread per node walks its root path.  The tree arrives in the launch arguments (768 bytes),
// so nothing has to be resident on the device beforehand.
__global__ void __launch_bounds__(MCSD_MAX_NODES)
build_mask_kernel(const __grid_constant__ TreeArg tree, int n_nodes, int words,
                  uint64_t* __restrict__ anc, int32_t* __restrict__ depth, int32_t* __restrict__ level_start) {
    __shared__ int s_depth[MCSD_MAX_NODES];
    const int n = threadIdx.x;
    if (n < n_nodes) {
        uint64_t bits[MCSD_MAX_WORDS] = {0, 0, 0};
        int d = -1;
        int a = n;
        // a root path has at most n_nodes nodes; the bound keeps the walk finite on any input
        for (int step = 0; a >= 0 && step < n_nodes; ++step) {
            bits[a >> 6] |= 1ull << (a & 63);
            ++d;
            a = tree.parent[a];
        }
        for (int w = 0; w < words; ++w) anc[(size_t)n * words + w] = (w < MCSD_MAX_WORDS) ? bits[w] : 0ull;
        depth[n] = d;
        s_depth[n] = d;
    }
    __syncthreads();
    if (level_start != nullptr && n < n_nodes) {
        if (n == 0 || s_depth[n - 1] != s_depth[n]) level_start[s_depth[n]] = n;
        if (n == n_nodes - 1) level_start[s_depth[n] + 1] = n_nodes;
    }
}

}  // namespace mcsd

extern "C" int mcsd_build_mask(const int32_t* parent_host, int n_nodes, uint64_t* anc_dev, int words,
                               int32_t* depth_dev, int32_t* level_start_dev, int32_t* level_start_host,
                               int* n_levels, void* stream) {
    if (parent_host == nullptr || anc_dev == nullptr || depth_dev == nullptr) return MCSD_ERR_NULL;
    if (n_nodes < 1 || n_nodes > MCSD_MAX_NODES) return MCSD_ERR_BAD_SHAPE;
    if (words < (n_nodes + 63) / 64 || words > MCSD_MAX_WORDS) return MCSD_ERR_BAD_SHAPE;

    // level order: node 0 is a root, parents come earlier and never decrease (children contiguous),
    // depth never decreases
    mcsd::TreeArg tree;
    int depth[MCSD_MAX_NODES];
    if (parent_host[0] != -1) return MCSD_ERR_NOT_BFS;
    for (int n = 0; n < n_nodes; ++n) {
        const int p = parent_host[n];
        if (p < -1 || p >= n) return MCSD_ERR_NOT_BFS;
        if (n > 0 && p < parent_host[n - 1]) return MCSD_ERR_NOT_BFS;
        depth[n] = (p < 0) ? 0 : depth[p] + 1;
        if (n > 0 && depth[n] < depth[n - 1]) return MCSD_ERR_NOT_BFS;
        tree.parent[n] = p;
    }
    for (int n = n_nodes; n < MCSD_MAX_NODES; ++n) tree.parent[n] = -1;
    const int levels = depth[n_nodes - 1] + 1;
    if (n_levels != nullptr) *n_levels = levels;
    if (level_start_host != nullptr) {
        for (int n = 0; n < n_nodes; ++n)
            if (n == 0 || depth[n] != depth[n - 1]) level_start_host[depth[n]] = n;
        level_start_host[levels] = n_nodes;
    }

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    mcsd::build_mask_kernel<<<1, MCSD_MAX_NODES, 0, s>>>(tree, n_nodes, words, anc_dev, depth_dev, level_start_dev);
    MCSD_CUDA_CHECK(cudaGetLastError());
    mcsd::count_launches(1);
    return MCSD_OK;
}
