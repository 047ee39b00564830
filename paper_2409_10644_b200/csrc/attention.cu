// C ABI entry point of tree attention (Section 2.2 of the paper): argument checks, workspace carving and
// the choice between the tcgen05 tensor-core kernel (bf16, head_dim 128) and the CUDA-core kernel.
#include "attention.cuh"

namespace mcsd {

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static bool use_tc(const AttentionArgs& a) {
    return a.dtype == MCSD_BF16 && a.D == 128 && aligned16(a.q) && aligned16(a.k_cache) && aligned16(a.v_cache) &&
           aligned16(a.k_tree) && aligned16(a.v_tree) && aligned16(a.out) && tc_supported(a);
}

}  // namespace mcsd

static int check_shape(int B, int H, int N, int D, int L_max, int dtype) {
    if (dtype != MCSD_BF16 && dtype != MCSD_F32) return MCSD_ERR_BAD_DTYPE;
    if (B < 1 || H < 1 || N < 1 || N > MCSD_MAX_NODES || L_max < 0) return MCSD_ERR_BAD_SHAPE;
    if (D != 64 && D != 128) return MCSD_ERR_BAD_SHAPE;
    if ((long long)B * H > 65535) return MCSD_ERR_BAD_SHAPE;
    return MCSD_OK;
}

extern "C" size_t mcsd_tree_attention_workspace_bytes(int B, int H, int N, int D, int L_max, int dtype) {
    if (check_shape(B, H, N, D, L_max, dtype) != MCSD_OK) return 0;
    size_t scratch = mcsd::simt_workspace_bytes(B, H, N, D, L_max);
    if (dtype == MCSD_BF16 && D == 128) {
        const size_t tc = mcsd::tc_workspace_bytes(B, H, N, D, L_max);
        if (tc > scratch) scratch = tc;
    }
    return sizeof(mcsd::WorkspaceHeader) + mcsd::align_up(scratch, 256);
}

static int run_attention(const void* q, const void* k_cache, const void* v_cache, const void* k_tree, const void* v_tree,
                         void* out, const int32_t* seq_lens, const int32_t* n_active, const uint64_t* anc, int words,
                         int B, int H, int G, int N, int D, int L_max, float softmax_scale, int dtype, void* workspace,
                         size_t workspace_bytes, void* stream) {
    if (!q || !k_tree || !v_tree || !out || !seq_lens || !anc || !workspace) return MCSD_ERR_NULL;
    const int st = check_shape(B, H, N, D, L_max, dtype);
    if (st != MCSD_OK) return st;
    if (G < 1 || H % G != 0) return MCSD_ERR_BAD_SHAPE;
    if (L_max > 0 && (!k_cache || !v_cache)) return MCSD_ERR_NULL;
    if (words < (N + 63) / 64 || words > MCSD_MAX_WORDS) return MCSD_ERR_BAD_SHAPE;
    if (workspace_bytes < mcsd_tree_attention_workspace_bytes(B, H, N, D, L_max, dtype))
        return MCSD_ERR_WORKSPACE_TOO_SMALL;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MCSD_ERR_BAD_SHAPE;

    mcsd::AttentionArgs a{q, k_cache, v_cache, k_tree, v_tree, out, seq_lens, n_active, anc, words,
                          B, H, N, D, L_max, softmax_scale, dtype, G};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    auto* header = static_cast<mcsd::WorkspaceHeader*>(workspace);
    void* scratch = static_cast<char*>(workspace) + sizeof(mcsd::WorkspaceHeader);
    const size_t scratch_bytes = workspace_bytes - sizeof(mcsd::WorkspaceHeader);
    if (mcsd::use_tc(a)) return mcsd::tree_attention_tc(a, header, scratch, scratch_bytes, s);
    return mcsd::tree_attention_simt(a, scratch, s);
}

extern "C" int mcsd_selftest_bounded_wait(void* workspace, size_t workspace_bytes, int microseconds, void* stream) {
    if (!workspace) return MCSD_ERR_NULL;
    if (workspace_bytes < sizeof(mcsd::WorkspaceHeader) || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MCSD_ERR_BAD_SHAPE;
    if (microseconds < 1 || microseconds > 100000) return MCSD_ERR_BAD_SHAPE;     // at most a tenth of a second
    // clock64 ticks at the SM clock, at most about 2 GHz: 2000 cycles per microsecond bound the wait from above
    return mcsd::tc_bounded_wait_selftest(static_cast<mcsd::WorkspaceHeader*>(workspace), 2000LL * microseconds, 42,
                                          static_cast<cudaStream_t>(stream));
}

extern "C" int mcsd_tree_attention_path(int B, int H_q, int H_kv, int N, int D, int L_max, int dtype) {
    const int st = check_shape(B, H_q, N, D, L_max, dtype);
    if (st != MCSD_OK) return st;
    if (H_kv < 1 || H_q < H_kv || H_q % H_kv != 0) return MCSD_ERR_BAD_SHAPE;
    return mcsd::tc_shape_supported(B, H_q, H_q / H_kv, N, D, L_max, dtype) ? MCSD_PATH_TENSOR_CORE : MCSD_PATH_CUDA_CORE;
}

extern "C" int mcsd_tree_attention_plan(int B, int H_q, int H_kv, int N, int D, int L_max, int dtype, const int32_t* seq_lens,
                                        const int32_t* n_active, int n_blocks, int64_t* first_tile, int64_t* info,
                                        int n_probe, const int64_t* probe_tiles, int64_t* probe_out) {
    const int path = mcsd_tree_attention_path(B, H_q, H_kv, N, D, L_max, dtype);
    if (path < 0) return path;
    if (path != MCSD_PATH_TENSOR_CORE) return MCSD_ERR_BAD_SHAPE;
    if (!seq_lens || !first_tile || (n_probe > 0 && (!probe_tiles || !probe_out))) return MCSD_ERR_NULL;
    if (n_blocks < 1 || n_blocks > mcsd::kTcMaxBlocks || n_probe < 0) return MCSD_ERR_BAD_SHAPE;
    static_assert(sizeof(long long) == sizeof(int64_t), "64-bit long long");
    return mcsd::tc_plan_host(B, H_q, H_q / H_kv, N, L_max, seq_lens, n_active, n_blocks, reinterpret_cast<long long*>(first_tile),
                              reinterpret_cast<long long*>(info), n_probe, reinterpret_cast<const long long*>(probe_tiles),
                              reinterpret_cast<long long*>(probe_out));
}

extern "C" int mcsd_tree_attention(const void* q, const void* k_cache, const void* v_cache, const void* k_tree,
                                   const void* v_tree, void* out, const int32_t* seq_lens, const int32_t* n_active,
                                   const uint64_t* anc, int words, int B, int H, int N, int D, int L_max,
                                   float softmax_scale, int dtype, void* workspace, size_t workspace_bytes,
                                   void* stream) {
    return run_attention(q, k_cache, v_cache, k_tree, v_tree, out, seq_lens, n_active, anc, words, B, H, 1, N, D, L_max,
                         softmax_scale, dtype, workspace, workspace_bytes, stream);
}

extern "C" int mcsd_tree_attention_gqa(const void* q, const void* k_cache, const void* v_cache, const void* k_tree,
                                       const void* v_tree, void* out, const int32_t* seq_lens, const int32_t* n_active,
                                       const uint64_t* anc, int words, int B, int H_q, int H_kv, int N, int D, int L_max,
                                       float softmax_scale, int dtype, void* workspace, size_t workspace_bytes,
                                       void* stream) {
    if (H_kv < 1 || H_q < H_kv || H_q % H_kv != 0) return MCSD_ERR_BAD_SHAPE;
    return run_attention(q, k_cache, v_cache, k_tree, v_tree, out, seq_lens, n_active, anc, words, B, H_q, H_q / H_kv, N,
                         D, L_max, softmax_scale, dtype, workspace, workspace_bytes, stream);
}
