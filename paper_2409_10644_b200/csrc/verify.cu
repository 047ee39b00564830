// Multi-candidate accept/reject over a token tree (Fig. 1 steps 4-6 of the paper; Section 3.1 for several
// target-initialised roots).
//
// The walk of one root visits a node, tries its children in order and either moves to the first accepted
// child or stops.  Uniforms are indexed by node, so what happens at a node does not depend on how the walk
// got there.  That splits the work in two kernels:
//
//   verify_nodes_kernel   one thread block per (sequence, node): decides which child, if any, is accepted
//                         at that node.  After m rejections the target-side distribution is
//                         max(p - c_m q, 0) / Y_m with c_0 = 0, Y_0 = 1, c_{m+1} = c_m + Y_m and
//                         Y_m = sum_v max(p_v - c_m q_v, 0): iterating norm(max(pt - q, 0)) never needs a
//                         vocabulary-sized write, only one reduction over the (p, q) rows per rejection.
//                         A node whose first child is accepted reads two scalars and no row at all.
//   verify_select_kernel  one thread block per sequence: follows next_child from every root, keeps the
//                         longest path (ties: lowest root), then draws the new token at its stop node by
//                         inverse CDF in token-id order and, on request, lists the most probable ids.
//
// Rows are read with 128-bit loads when the row length allows; reductions run in a fixed order, fp32 per
// lane and fp64 across warps.
#include <mutex>

#include "common.cuh"

namespace mcsd {

constexpr int kVerifyThreads = 1024;
constexpr int kVerifyWarps = kVerifyThreads / 32;

struct NodeState {
    int32_t next_child;   // accepted child, or -1 if the walk stops here
    int32_t pad;
    double c;             // stop distribution is max(p - c q, 0); c = 0 means the row p itself
};

__device__ __forceinline__ float4 load4(const float* __restrict__ row, int idx, int V, bool vec) {
    if (vec) return __ldg(reinterpret_cast<const float4*>(row + idx));
    float4 r;
    r.x = idx + 0 < V ? __ldg(row + idx + 0) : 0.f;
    r.y = idx + 1 < V ? __ldg(row + idx + 1) : 0.f;
    r.z = idx + 2 < V ? __ldg(row + idx + 2) : 0.f;
    r.w = idx + 3 < V ? __ldg(row + idx + 3) : 0.f;
    return r;
}

__device__ __forceinline__ float4 residual4(const float* __restrict__ p, const float* __restrict__ q, float c,
                                            int idx, int V, bool vec) {
    float4 a = load4(p, idx, V, vec);
    if (c != 0.f) {
        const float4 b = load4(q, idx, V, vec);
        a.x = fmaxf(fmaf(-c, b.x, a.x), 0.f);
        a.y = fmaxf(fmaf(-c, b.y, a.y), 0.f);
        a.z = fmaxf(fmaf(-c, b.z, a.z), 0.f);
        a.w = fmaxf(fmaf(-c, b.w, a.w), 0.f);
    }
    return a;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// sum_v max(p_v - c q_v, 0) over one row, same value in every thread of the block
__device__ double residual_mass(const float* __restrict__ p, const float* __restrict__ q, float c, int V, bool vec,
                                double* s_warp) {
    float acc = 0.f;
    for (int idx = threadIdx.x * 4; idx < V; idx += kVerifyThreads * 4) {
        const float4 r = residual4(p, q, c, idx, V, vec);
        acc += (r.x + r.y) + (r.z + r.w);
    }
    acc = warp_sum(acc);
    __syncthreads();                       // s_warp may still be read from a previous call
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = (double)acc;
    __syncthreads();
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < kVerifyWarps; ++w) tot += s_warp[w];
    return tot;
}

__device__ __forceinline__ int active_nodes(const int32_t* gamma, const int32_t* level_start, int n_levels, int b, int N) {
    if (gamma == nullptr) return N;
    int g = gamma[b];
    g = g < 0 ? 0 : (g > n_levels - 1 ? n_levels - 1 : g);
    return min(level_start[g + 1], N);
}

__global__ void __launch_bounds__(kVerifyThreads)
verify_nodes_kernel(const float* __restrict__ p, const float* __restrict__ q, const int32_t* __restrict__ tokens,
                    const int32_t* __restrict__ parent, const int32_t* __restrict__ level_start, int n_levels,
                    const int32_t* __restrict__ gamma, const float* __restrict__ u_accept,
                    int N, int V, NodeState* __restrict__ state) {
    __shared__ int s_first, s_cnt, s_accept;
    __shared__ double s_warp[kVerifyWarps];
    const int b = blockIdx.y, u = blockIdx.x, tid = threadIdx.x;
    const int n_act = active_nodes(gamma, level_start, n_levels, b, N);
    if (u >= n_act) return;
    if (tid == 0) { s_first = N; s_cnt = 0; }
    __syncthreads();
    for (int c = tid; c < N; c += kVerifyThreads)
        if (parent[c] == u) { atomicMin(&s_first, c); atomicAdd(&s_cnt, 1); }
    __syncthreads();
    const int first = s_first, cnt = s_cnt;

    NodeState st;
    st.next_child = -1; st.pad = 0; st.c = 0.0;
    // in level order a kept prefix of the tree keeps either all children of a node or none
    if (cnt > 0 && first < n_act) {
        const float* pr = p + ((size_t)b * N + u) * V;
        const float* qr = q + ((size_t)b * N + u) * V;
        const bool vec = (V % 4 == 0) && ((reinterpret_cast<uintptr_t>(pr) | reinterpret_cast<uintptr_t>(qr)) % 16 == 0);
        double c = 0.0, Y = 1.0;
        for (int m = 0; m < cnt; ++m) {
            const int child = first + m;
            if (tid == 0) {
                const int x = tokens[(size_t)b * N + child];
                double a = 0.0;
                if (x >= 0 && x < V) {
                    const double px = (double)pr[x], qx = (double)qr[x];
                    const double num = fmax(px - c * qx, 0.0);
                    a = qx > 0.0 ? fmin(1.0, num / (Y * qx)) : (num > 0.0 ? 1.0 : 0.0);
                }
                s_accept = ((double)u_accept[(size_t)b * N + child] < a) ? 1 : 0;
            }
            __syncthreads();
            const int acc = s_accept;
            __syncthreads();
            if (acc) { st.next_child = child; break; }
            c += Y;
            Y = residual_mass(pr, qr, (float)c, V, vec, s_warp);
            if (!(Y > 0.0)) { c = 0.0; Y = 1.0; }     // nothing left: back to the un-residualised row
        }
        if (st.next_child < 0) st.c = c;
    }
    if (tid == 0) state[(size_t)b * N + u] = st;
}

// (value, id) order used for the list of most probable ids: larger value first, ties to the smaller id
__device__ __forceinline__ bool better(float va, int ia, float vb, int ib) {
    return va > vb || (va == vb && ia < ib);
}

__global__ void __launch_bounds__(kVerifyThreads)
verify_select_kernel(const float* __restrict__ p, const float* __restrict__ q, const int32_t* __restrict__ tokens,
                     const NodeState* __restrict__ state, int n_levels, int n_roots,
                     const float* __restrict__ u_bonus, int N, int V,
                     int32_t* __restrict__ accept_len, int32_t* __restrict__ out_tokens,
                     int32_t* __restrict__ out_nodes, int32_t* __restrict__ best_root,
                     int32_t* __restrict__ next_roots, int R) {
    __shared__ int s_len[MCSD_MAX_NODES];
    __shared__ int s_stop, s_slot;
    __shared__ double s_tot[kVerifyWarps];
    __shared__ int s_last[kVerifyWarps];
    __shared__ float s_bv[kVerifyWarps];
    __shared__ int s_bi[kVerifyWarps];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const NodeState* st = state + (size_t)b * N;

    if (tid < n_roots) {
        int u = tid, len = 0;
        for (int step = 0; step < n_levels; ++step) {
            const int nc = st[u].next_child;
            if (nc < 0 || nc >= N) break;
            u = nc;
            ++len;
        }
        s_len[tid] = len;
    }
    __syncthreads();
    if (tid == 0) {
        int best = 0;
        for (int r = 1; r < n_roots; ++r)
            if (s_len[r] > s_len[best]) best = r;
        int32_t* ot = out_tokens + (size_t)b * (n_levels + 1);
        int32_t* on = out_nodes + (size_t)b * n_levels;
        for (int i = 0; i < n_levels + 1; ++i) ot[i] = -1;
        for (int i = 0; i < n_levels; ++i) on[i] = -1;
        int slot = 0;
        if (n_roots > 1) ot[slot++] = tokens[(size_t)b * N + best];
        int u = best;
        for (int i = 0; i < s_len[best]; ++i) {
            u = st[u].next_child;
            on[i] = u;
            ot[slot++] = tokens[(size_t)b * N + u];
        }
        accept_len[b] = s_len[best];
        best_root[b] = best;
        s_stop = u;
        s_slot = slot;
    }
    __syncthreads();
    const int u = s_stop;
    const float c = (float)st[u].c;
    const float* pr = p + ((size_t)b * N + u) * V;
    const float* qr = q + ((size_t)b * N + u) * V;
    const bool vec = (V % 4 == 0) && ((reinterpret_cast<uintptr_t>(pr) | reinterpret_cast<uintptr_t>(qr)) % 16 == 0);

    // ---- new token: inverse CDF over dist_v = max(p_v - c q_v, 0) in token-id order ----
    // pass 1: every warp sums one contiguous range of ids
    const int span = ((V + kVerifyWarps - 1) / kVerifyWarps + 127) / 128 * 128;
    {
        const int lo = warp * span, hi = min(V, lo + span);
        float acc = 0.f;
        int last = -1;
        for (int idx = lo + lane * 4; idx < hi; idx += 128) {
            const float4 r = residual4(pr, qr, c, idx, V, vec);
            acc += (r.x + r.y) + (r.z + r.w);
            if (r.x > 0.f) last = idx;
            if (r.y > 0.f) last = idx + 1;
            if (r.z > 0.f) last = idx + 2;
            if (r.w > 0.f) last = idx + 3;
        }
        acc = warp_sum(acc);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
        if (lane == 0) { s_tot[warp] = (double)acc; s_last[warp] = last; }
    }
    __syncthreads();
    // pass 2: one warp locates the crossing, starting in the range where the running sum passes u * Z
    if (warp == 0) {
        double total = 0.0;
        int last_pos = -1;
        for (int w = 0; w < kVerifyWarps; ++w) { total += s_tot[w]; last_pos = max(last_pos, s_last[w]); }
        const double target = (double)u_bonus[(size_t)b * N + u] * total;
        double base = 0.0;
        int w0 = 0;
        while (w0 < kVerifyWarps && !(base + s_tot[w0] > target)) { base += s_tot[w0]; ++w0; }
        int found = -1;
        for (int w = w0; w < kVerifyWarps && found < 0; ++w) {
            const int lo = w * span, hi = min(V, lo + span);
            for (int i0 = lo; i0 < hi && found < 0; i0 += 128) {
                const int idx = i0 + lane * 4;
                float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
                if (idx < hi) r = residual4(pr, qr, c, idx, V, vec);
                const float ls = (r.x + r.y) + (r.z + r.w);
                float incl = ls;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += t;
                }
                const bool hit = (base + (double)incl > target) && idx < hi;
                const unsigned ballot = __ballot_sync(0xffffffffu, hit);
                if (ballot != 0u) {
                    const int L = __ffs(ballot) - 1;
                    int tok = -1;
                    if (lane == L) {
                        const double ex = base + (double)(incl - ls);
                        const float e1 = r.x, e2 = r.x + r.y, e3 = (r.x + r.y) + r.z;
                        if (ex + (double)e1 > target) tok = idx;
                        else if (ex + (double)e2 > target) tok = idx + 1;
                        else if (ex + (double)e3 > target) tok = idx + 2;
                        else tok = idx + 3;
                        if (tok >= V) tok = V - 1;
                    }
                    found = __shfl_sync(0xffffffffu, tok, L);
                } else {
                    base += (double)__shfl_sync(0xffffffffu, incl, 31);
                }
            }
        }
        if (found < 0) found = last_pos >= 0 ? last_pos : V - 1;
        if (lane == 0) out_tokens[(size_t)b * (n_levels + 1) + s_slot] = found;
    }

    // ---- optional: the R most probable ids of the same distribution ----
    if (next_roots != nullptr && R > 0) {
        float pv = __int_as_float(0x7f800000);   // previous pick: +inf, id -1
        int pi = -1;
        for (int r = 0; r < R; ++r) {
            float bv = -1.f;
            int bi = -1;
            for (int idx = tid * 4; idx < V; idx += kVerifyThreads * 4) {
                const float4 e = residual4(pr, qr, c, idx, V, vec);
                const float ev[4] = {e.x, e.y, e.z, e.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int id = idx + k;
                    if (id < V && better(pv, pi, ev[k], id) && (bi < 0 || better(ev[k], id, bv, bi))) { bv = ev[k]; bi = id; }
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (oi >= 0 && (bi < 0 || better(ov, oi, bv, bi))) { bv = ov; bi = oi; }
            }
            __syncthreads();
            if (lane == 0) { s_bv[warp] = bv; s_bi[warp] = bi; }
            __syncthreads();
            bv = s_bv[0]; bi = s_bi[0];
            for (int w = 1; w < kVerifyWarps; ++w)
                if (s_bi[w] >= 0 && (bi < 0 || better(s_bv[w], s_bi[w], bv, bi))) { bv = s_bv[w]; bi = s_bi[w]; }
            if (tid == 0) next_roots[(size_t)b * R + r] = bi;
            pv = bv; pi = bi;
            if (bi < 0) {                       // fewer than R ids in the vocabulary
                for (int rr = r + 1 + tid; rr < R; rr += kVerifyThreads) next_roots[(size_t)b * R + rr] = -1;
                break;
            }
        }
    }
}

}  // namespace mcsd

extern "C" size_t mcsd_verify_tree_workspace_bytes(int B, int N, int V) {
    (void)V;
    if (B < 1 || N < 1) return 0;
    return mcsd::align_up(sizeof(mcsd::WorkspaceHeader) + sizeof(mcsd::NodeState) * (size_t)B * N, 256);
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
    mcsd::verify_nodes_kernel<<<dim3(N, B), mcsd::kVerifyThreads, 0, s>>>(p, q, tokens, parent, level_start, n_levels,
                                                                        gamma, u_accept, N, V, state);
    MCSD_CUDA_CHECK(cudaGetLastError());
    mcsd::verify_select_kernel<<<B, mcsd::kVerifyThreads, 0, s>>>(p, q, tokens, state, n_levels, n_roots, u_bonus, N, V,
                                                                 accept_len, out_tokens, out_nodes, best_root,
                                                                 R > 0 ? next_roots : nullptr, R);
    MCSD_CUDA_CHECK(cudaGetLastError());
    mcsd::count_launches(2);
    return MCSD_OK;
}

// ------------------------------------------------------------------------------------------------------
// Variant with built-in scratch, for callers that cannot allocate device memory.
// ------------------------------------------------------------------------------------------------------
namespace mcsd {

// Scratch that lives in the library image itself: one copy per GPU that loads the library, held until the
// process exits.  Layout: workspace header, then MCSD_STATIC_VERIFY_MAX_STATES node states.
constexpr size_t kStaticScratchBytes = sizeof(WorkspaceHeader) + sizeof(NodeState) * (size_t)MCSD_STATIC_VERIFY_MAX_STATES;
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
    // the array keeps whatever the previous call left; the status line must start at zero
    MCSD_CUDA_CHECK(cudaMemsetAsync(scratch, 0, sizeof(mcsd::WorkspaceHeader), static_cast<cudaStream_t>(stream)));
    return mcsd_verify_tree(p, q, tokens, parent, level_start, n_levels, n_roots, gamma, u_accept, u_bonus, B, N, V,
                            accept_len, out_tokens, out_nodes, best_root, next_roots, R, scratch,
                            mcsd::kStaticScratchBytes, stream);
}
