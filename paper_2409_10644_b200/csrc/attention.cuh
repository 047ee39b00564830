// Internal interface between the C ABI entry point of tree attention and its kernels.
#pragma once

#include "common.cuh"

namespace mcsd {

struct AttentionArgs {
    const void* q;
    const void* k_cache;
    const void* v_cache;
    const void* k_tree;
    const void* v_tree;
    void* out;
    const int32_t* seq_lens;
    const int32_t* n_active;
    const uint64_t* anc;
    int words;
    int B, H, N, D, L_max;   // H: query heads
    float scale;
    int dtype;
    int G;                   // query heads per key/value head (1: multi-head attention); key/value tensors have H / G heads
};

// CUDA-core path (fp32, or bf16 shapes the tensor-core kernel does not take)
size_t simt_workspace_bytes(int B, int H, int N, int D, int L_max);
int tree_attention_simt(const AttentionArgs& a, void* scratch, cudaStream_t stream);

// tcgen05 tensor-core path: bf16, D = 128
bool tc_shape_supported(int B, int H, int G, int N, int D, int L_max, int dtype);   // shape and dtype alone
bool tc_supported(const AttentionArgs& a);
size_t tc_workspace_bytes(int B, int H, int N, int D, int L_max);
int tc_bounded_wait_selftest(WorkspaceHeader* header, long long limit_cycles, int where, cudaStream_t stream);
int tc_plan_host(int B, int H, int G, int N, int L_max, const int32_t* seq_lens, const int32_t* n_active, int grid,
                 long long* first_tile, long long* info, int n_probe, const long long* probe_tiles, long long* probe_out);
constexpr int kTcMaxBlocks = 160;                    // thread blocks of a launch, at most (one per multiprocessor)
int tree_attention_tc(const AttentionArgs& a, WorkspaceHeader* header, void* scratch, size_t scratch_bytes,
                      cudaStream_t stream);

}  // namespace mcsd
