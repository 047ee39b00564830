// Tensor-core path of tree attention; not built yet: every shape takes the CUDA-core kernel.
#include "attention.cuh"
namespace mcsd {
bool tc_supported(const AttentionArgs&) { return false; }
size_t tc_workspace_bytes(int, int, int, int, int) { return 0; }
int tree_attention_tc(const AttentionArgs&, WorkspaceHeader*, void*, size_t, cudaStream_t) { return MCSD_ERR_BAD_DTYPE; }
}  // namespace mcsd
