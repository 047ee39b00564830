// Multi-candidate accept/reject straight from next-token logits (Fig. 1 step 4, where logits become the
// distributions that are compared) at the two sampling settings of Section 4.1:
//
//   temperature > 0   p = softmax(target logits / T), q = softmax(draft logits / T); the accept/reject kernels of
//                     verify_kernels.cuh run on logit rows, so p and q are never written to memory.
//   temperature == 0  greedy: the target distribution is the point mass on its largest logit, a candidate is
//                     accepted iff it is that token, and the new token is the largest logit of the stop node.
#include "verify_kernels.cuh"

namespace mcsd {

// one thread block per (sequence, node): id of the largest target logit (ties: lowest id) and the first child
// that carries it
template <typename T>
__global__ void __launch_bounds__(kVerifyThreads)
greedy_nodes_kernel(const T* __restrict__ zt, const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                    const int32_t* __restrict__ level_start, int n_levels, const int32_t* __restrict__ gamma,
                    int N, int V, NodeState* __restrict__ state) {
    constexpr int E = LogitLoad<T>::E;
    __shared__ int s_first, s_cnt;
    __shared__ float s_bv[kVerifyWarps];
    __shared__ int s_bi[kVerifyWarps];
    const int b = blockIdx.y, u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_act = active_nodes(gamma, level_start, n_levels, b, N);
    if (u >= n_act) return;
    int first, cnt;
    find_children(parent, u, N, &s_first, &s_cnt, first, cnt);

    const T* row = zt + ((size_t)b * N + u) * V;
    const bool vec = (V % E == 0) && (reinterpret_cast<uintptr_t>(row) % 16 == 0);
    float bv = 0.f;
    int bi = -1;
    int idx = tid * E;
    if (vec) {                                   // several steps' loads in flight at once, compared in id order
        constexpr int kStep = kVerifyThreads * E;
        for (; idx + (kRowBatch - 1) * kStep < V; idx += kRowBatch * kStep) {
            float a[kRowBatch][E];
#pragma unroll
            for (int j = 0; j < kRowBatch; ++j) LogitLoad<T>::load_vec(row, idx + j * kStep, a[j]);
#pragma unroll
            for (int j = 0; j < kRowBatch; ++j)
#pragma unroll
                for (int i = 0; i < E; ++i)
                    if (bi < 0 || a[j][i] > bv) { bv = a[j][i]; bi = idx + j * kStep + i; }
        }
    }
    for (; idx < V; idx += kVerifyThreads * E) {
        float a[E];
        LogitLoad<T>::load(row, idx, V, vec, a);
#pragma unroll
        for (int i = 0; i < E; ++i)
            if (idx + i < V && (bi < 0 || a[i] > bv)) { bv = a[i]; bi = idx + i; }   // ids ascend: '>' keeps the lowest
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (oi >= 0 && (bi < 0 || better(ov, oi, bv, bi))) { bv = ov; bi = oi; }
    }
    if (lane == 0) { s_bv[warp] = bv; s_bi[warp] = bi; }
    __syncthreads();
    if (tid == 0) {
        bv = s_bv[0]; bi = s_bi[0];
        for (int w = 1; w < kVerifyWarps; ++w)
            if (s_bi[w] >= 0 && (bi < 0 || better(s_bv[w], s_bi[w], bv, bi))) { bv = s_bv[w]; bi = s_bi[w]; }
        NodeState st;
        st.next_child = -1; st.top = bi; st.c = 0.0;
        // in level order a kept prefix of the tree keeps either all children of a node or none
        if (cnt > 0 && first < n_act) {
            for (int m = 0; m < cnt; ++m)
                if (tokens[(size_t)b * N + first + m] == bi) { st.next_child = first + m; break; }
        }
        state[(size_t)b * N + u] = st;
    }
}

// one thread block per sequence: longest path, new token = largest logit of the stop node, optional list of
// the R largest logits there
template <typename T>
__global__ void __launch_bounds__(kVerifyThreads)
greedy_select_kernel(const T* __restrict__ zt, const int32_t* __restrict__ tokens, const NodeState* __restrict__ state,
                     int n_levels, int n_roots, int N, int V, int32_t* __restrict__ accept_len,
                     int32_t* __restrict__ out_tokens, int32_t* __restrict__ out_nodes,
                     int32_t* __restrict__ best_root, int32_t* __restrict__ next_roots, int R) {
    constexpr int E = LogitLoad<T>::E;
    __shared__ int s_len[MCSD_MAX_NODES];
    __shared__ int s_stop, s_slot;
    __shared__ float s_bv[kVerifyWarps];
    __shared__ int s_bi[kVerifyWarps];
    const int b = blockIdx.x;
    const NodeState* st = state + (size_t)b * N;
    select_path(st, tokens, b, n_levels, n_roots, N, accept_len, out_tokens, out_nodes, best_root, s_len, &s_stop, &s_slot);
    const int u = s_stop;
    if (threadIdx.x == 0) out_tokens[(size_t)b * (n_levels + 1) + s_slot] = st[u].top;
    if (next_roots != nullptr && R > 0) {
        const T* row = zt + ((size_t)b * N + u) * V;
        const bool vec = (V % E == 0) && (reinterpret_cast<uintptr_t>(row) % 16 == 0);
        auto load = [row, V, vec](int idx, float (&r)[E]) { LogitLoad<T>::load(row, idx, V, vec, r); };
        top_ids<E>(load, V, R, next_roots + (size_t)b * R, s_bv, s_bi);
    }
}

template <typename T>
static int launch_logits(const void* target_logits, const void* draft_logits, float temperature, const int32_t* tokens,
                         const int32_t* parent, const int32_t* level_start, int n_levels, int n_roots,
                         const int32_t* gamma, const float* u_accept, const float* u_bonus, int B, int N, int V,
                         int32_t* accept_len, int32_t* out_tokens, int32_t* out_nodes, int32_t* best_root,
                         int32_t* next_roots, int R, NodeState* state, int* tickets, cudaStream_t s) {
    const T* zt = static_cast<const T*>(target_logits);
    if (temperature == 0.f) {
        greedy_nodes_kernel<T><<<dim3(N, B), kVerifyThreads, 0, s>>>(zt, tokens, parent, level_start, n_levels, gamma, N, V,
                                                                    state);
        MCSD_CUDA_CHECK(cudaGetLastError());
        greedy_select_kernel<T><<<B, kVerifyThreads, 0, s>>>(zt, tokens, state, n_levels, n_roots, N, V, accept_len,
                                                            out_tokens, out_nodes, best_root, next_roots, R);
        MCSD_CUDA_CHECK(cudaGetLastError());
        count_launches(2);
    } else {
        const LogitRows<T> rows{zt, static_cast<const T*>(draft_logits), 1.4426950408889634f / temperature};
        verify_tree_kernel<LogitRows<T>><<<dim3(N, B), kVerifyThreads, 0, s>>>(
            rows, tokens, parent, level_start, n_levels, n_roots, gamma, u_accept, u_bonus, N, V, state, tickets, accept_len,
            out_tokens, out_nodes, best_root, next_roots, R);
        MCSD_CUDA_CHECK(cudaGetLastError());
        count_launches(1);
    }
    return MCSD_OK;
}

}  // namespace mcsd

extern "C" int mcsd_verify_tree_logits(const void* target_logits, const void* draft_logits, int dtype, float temperature,
                                       const int32_t* tokens, const int32_t* parent, const int32_t* level_start,
                                       int n_levels, int n_roots, const int32_t* gamma, const float* u_accept,
                                       const float* u_bonus, int B, int N, int V, int32_t* accept_len,
                                       int32_t* out_tokens, int32_t* out_nodes, int32_t* best_root,
                                       int32_t* next_roots, int R, void* workspace, size_t workspace_bytes,
                                       void* stream) {
    if (!target_logits || !tokens || !parent || !level_start || !accept_len || !out_tokens || !out_nodes ||
        !best_root || !workspace)
        return MCSD_ERR_NULL;
    if (!(temperature >= 0.f) || !(temperature <= 1e6f)) return MCSD_ERR_BAD_SHAPE;      // also rejects NaN
    if (temperature > 0.f && temperature < 1e-3f) return MCSD_ERR_BAD_SHAPE;
    if (temperature > 0.f && (!draft_logits || !u_accept || !u_bonus)) return MCSD_ERR_NULL;
    if (dtype != MCSD_BF16 && dtype != MCSD_F32) return MCSD_ERR_BAD_DTYPE;
    if (B < 1 || N < 1 || V < 1 || N > MCSD_MAX_NODES || B > 65535) return MCSD_ERR_BAD_SHAPE;
    if (n_levels < 1 || n_levels > N || n_roots < 1 || n_roots > N) return MCSD_ERR_BAD_SHAPE;
    if (R < 0 || R > 32) return MCSD_ERR_BAD_SHAPE;
    if (R > 0 && !next_roots) return MCSD_ERR_NULL;
    if (workspace_bytes < mcsd_verify_tree_workspace_bytes(B, N, V)) return MCSD_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    auto* state = reinterpret_cast<mcsd::NodeState*>(static_cast<char*>(workspace) + sizeof(mcsd::WorkspaceHeader));
    int* tickets = reinterpret_cast<int*>(static_cast<char*>(workspace) + mcsd::verify_tickets_offset(B, N));
    int32_t* roots = R > 0 ? next_roots : nullptr;
    if (dtype == MCSD_F32)
        return mcsd::launch_logits<float>(target_logits, draft_logits, temperature, tokens, parent, level_start, n_levels,
                                          n_roots, gamma, u_accept, u_bonus, B, N, V, accept_len, out_tokens, out_nodes,
                                          best_root, roots, R, state, tickets, s);
    return mcsd::launch_logits<__nv_bfloat16>(target_logits, draft_logits, temperature, tokens, parent, level_start,
                                              n_levels, n_roots, gamma, u_accept, u_bonus, B, N, V, accept_len, out_tokens,
                                              out_nodes, best_root, roots, R, state, tickets, s);
}

extern "C" int mcsd_sample_roots_logits(const void* target_logits, const void* draft_logits, int dtype, float temperature,
                                        const int32_t* accept_len, const int32_t* out_nodes, const int32_t* best_root,
                                        int n_levels, const float* u_roots, int B, int N, int V, int R,
                                        int32_t* next_roots, const void* workspace, size_t workspace_bytes,
                                        void* stream) {
    if (!target_logits || !draft_logits || !accept_len || !out_nodes || !best_root || !u_roots || !next_roots ||
        !workspace)
        return MCSD_ERR_NULL;
    if (!(temperature >= 1e-3f) || !(temperature <= 1e6f)) return MCSD_ERR_BAD_SHAPE;      // also rejects NaN and 0
    if (dtype != MCSD_BF16 && dtype != MCSD_F32) return MCSD_ERR_BAD_DTYPE;
    if (B < 1 || N < 1 || V < 1 || N > MCSD_MAX_NODES || B > 65535) return MCSD_ERR_BAD_SHAPE;
    if (n_levels < 1 || n_levels > N || R < 1 || R > 32) return MCSD_ERR_BAD_SHAPE;
    if (workspace_bytes < mcsd_verify_tree_workspace_bytes(B, N, V)) return MCSD_ERR_WORKSPACE_TOO_SMALL;
    const auto* state = reinterpret_cast<const mcsd::NodeState*>(static_cast<const char*>(workspace) +
                                                                sizeof(mcsd::WorkspaceHeader));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const float k = 1.4426950408889634f / temperature;
    if (dtype == MCSD_F32) {
        const mcsd::LogitRows<float> rows{static_cast<const float*>(target_logits), static_cast<const float*>(draft_logits), k};
        mcsd::sample_roots_kernel<mcsd::LogitRows<float>><<<B, mcsd::kVerifyThreads, 0, s>>>(
            rows, state, accept_len, out_nodes, best_root, n_levels, u_roots, N, V, R, next_roots);
    } else {
        const mcsd::LogitRows<__nv_bfloat16> rows{static_cast<const __nv_bfloat16*>(target_logits),
                                                  static_cast<const __nv_bfloat16*>(draft_logits), k};
        mcsd::sample_roots_kernel<mcsd::LogitRows<__nv_bfloat16>><<<B, mcsd::kVerifyThreads, 0, s>>>(
            rows, state, accept_len, out_nodes, best_root, n_levels, u_roots, N, V, R, next_roots);
    }
    MCSD_CUDA_CHECK(cudaGetLastError());
    mcsd::count_launches(1);
    return MCSD_OK;
}
