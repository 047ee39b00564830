// Shared host-side helpers of libmcsd: status codes, CUDA error capture, workspace header.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "mcsd.h"

namespace mcsd {

// First bytes of every workspace: written by kernels, read by mcsd_workspace_status().
struct WorkspaceHeader {
    int32_t status;        // 0 or MCSD_ERR_TIMEOUT
    int32_t detail;        // where a bounded wait gave up (kernel-specific code)
    int32_t pad[62];
};
static_assert(sizeof(WorkspaceHeader) == 256, "workspace header is one 256-byte line");

void set_last_cuda_error(cudaError_t e);
void count_launches(int n);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace mcsd

#define MCSD_CUDA_CHECK(expr)                                  \
    do {                                                       \
        cudaError_t _e = (expr);                               \
        if (_e != cudaSuccess) {                               \
            ::mcsd::set_last_cuda_error(_e);                   \
            return MCSD_ERR_CUDA;                              \
        }                                                      \
    } while (0)
