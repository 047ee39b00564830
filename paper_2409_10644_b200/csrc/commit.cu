// KV-cache update after acceptance (Fig. 1 step 6 of the paper): the keys/values of the winning root and of the
// accepted tree tokens are appended to the prefix cache of every layer, and the prefix lengths grow accordingly.
// One launch covers all layers; it moves (1 + accepted) rows of 2*D*elt bytes per (layer, sequence, head), so it
// is latency-bound: 16-byte copies, one thread block per (sequence, head, layer).
#include "common.cuh"

namespace mcsd {

constexpr int kCommitThreads = 128;

// grid: (B * H, n_layers)
__global__ void __launch_bounds__(kCommitThreads)
commit_kv_kernel(void* const* __restrict__ k_cache_layers, void* const* __restrict__ v_cache_layers,
                 const void* const* __restrict__ k_tree_layers, const void* const* __restrict__ v_tree_layers,
                 const int32_t* __restrict__ seq_lens, const int32_t* __restrict__ accept_len,
                 const int32_t* __restrict__ out_nodes, const int32_t* __restrict__ best_root,
                 int n_levels, int H, int N, int L_max, int row_bytes) {
    const int bh = blockIdx.x, b = bh / H, layer = blockIdx.y;
    const int L = min(max(seq_lens[b], 0), L_max);
    const int acc = min(max(accept_len[b], 0), n_levels);
    const int count = min(1 + acc, L_max - L);                 // rows that still fit
    const int vec_per_row = row_bytes / 16;
    const uint4* kt = static_cast<const uint4*>(k_tree_layers[layer]) + (size_t)bh * N * vec_per_row;
    const uint4* vt = static_cast<const uint4*>(v_tree_layers[layer]) + (size_t)bh * N * vec_per_row;
    uint4* kc = static_cast<uint4*>(k_cache_layers[layer]) + ((size_t)bh * L_max + L) * vec_per_row;
    uint4* vc = static_cast<uint4*>(v_cache_layers[layer]) + ((size_t)bh * L_max + L) * vec_per_row;
    for (int idx = threadIdx.x; idx < count * vec_per_row; idx += kCommitThreads) {
        const int i = idx / vec_per_row, c = idx % vec_per_row;
        int node = i == 0 ? best_root[b] : out_nodes[(size_t)b * n_levels + (i - 1)];
        if (node < 0 || node >= N) continue;                    // malformed verify output: leave the row alone
        kc[(size_t)i * vec_per_row + c] = kt[(size_t)node * vec_per_row + c];
        vc[(size_t)i * vec_per_row + c] = vt[(size_t)node * vec_per_row + c];
    }
}

__global__ void bump_lens_kernel(int32_t* __restrict__ seq_lens, const int32_t* __restrict__ accept_len, int n_levels,
                                 int B, int L_max) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int L = min(max(seq_lens[b], 0), L_max);
    const int acc = min(max(accept_len[b], 0), n_levels);
    seq_lens[b] = min(L_max, L + 1 + acc);
}

}  // namespace mcsd

extern "C" int mcsd_commit_kv(void* const* k_cache_layers, void* const* v_cache_layers,
                              const void* const* k_tree_layers, const void* const* v_tree_layers, int n_layers,
                              int32_t* seq_lens, const int32_t* accept_len, const int32_t* out_nodes,
                              const int32_t* best_root, int n_levels, int B, int H, int N, int D, int L_max, int dtype,
                              void* stream) {
    if (!k_cache_layers || !v_cache_layers || !k_tree_layers || !v_tree_layers || !seq_lens || !accept_len ||
        !out_nodes || !best_root)
        return MCSD_ERR_NULL;
    if (dtype != MCSD_BF16 && dtype != MCSD_F32) return MCSD_ERR_BAD_DTYPE;
    if (n_layers < 1 || n_layers > 65535 || B < 1 || H < 1 || N < 1 || N > MCSD_MAX_NODES || L_max < 1 || n_levels < 1 ||
        n_levels > N)
        return MCSD_ERR_BAD_SHAPE;
    if (D != 64 && D != 128) return MCSD_ERR_BAD_SHAPE;
    const int row_bytes = D * (dtype == MCSD_F32 ? 4 : 2);      // a multiple of 16 for every supported shape
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    mcsd::commit_kv_kernel<<<dim3(B * H, n_layers), mcsd::kCommitThreads, 0, s>>>(
        k_cache_layers, v_cache_layers, k_tree_layers, v_tree_layers, seq_lens, accept_len, out_nodes, best_root,
        n_levels, H, N, L_max, row_bytes);
    MCSD_CUDA_CHECK(cudaGetLastError());
    mcsd::bump_lens_kernel<<<(B + 127) / 128, 128, 0, s>>>(seq_lens, accept_len, n_levels, B, L_max);
    MCSD_CUDA_CHECK(cudaGetLastError());
    mcsd::count_launches(2);
    return MCSD_OK;
}
