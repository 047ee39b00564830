// Multi-candidate accept/reject (Fig. 1 steps 4-6 of the paper) with the vocabulary split over several GPUs:
// every rank holds columns [v0, v0 + Vs) of the two probability tensors, as a tensor-parallel output layer
// leaves them.  The procedure and its results are those of mcsd_verify_tree; only three kinds of numbers have to
// cross ranks, all of them a few bytes per node, and the caller exchanges them between the launches:
//
//   1. p_u(x), q_u(x) of every candidate token x            (one owner per token: sum over ranks)
//   2. Y = sum_v max(p_v - c q_v, 0) after a rejection       (partial sums: sum over ranks), once per round
//   3. the mass of the stop distribution per rank            (gathered), then the new token (max over ranks)
//
// The walk state of a node (how many siblings were rejected, c, Y) is recomputed identically on every rank from
// the reduced numbers, so ranks never disagree about which rows still need a pass.  A round tests at most one
// sibling per node, so a tree whose nodes have at most k children takes k + 1 round launches.
#include "verify_kernels.cuh"

namespace mcsd {

struct ShardAux {
    int32_t stage;        // siblings rejected so far; -1 once the node is decided
    int32_t pending;      // a residual-mass pass was issued last round and its reduced sum is waiting
    double c;             // running residual coefficient
    double Y;             // mass of the current residual
};

struct ShardPick {
    int32_t stop;         // node the winning path stopped at
    int32_t slot;         // position of the new token in out_tokens
};

struct ShardLayout {
    NodeState* state;
    ShardAux* aux;
    ShardPick* pick;
};

static size_t shard_workspace_bytes(int B, int N) {
    size_t n = sizeof(WorkspaceHeader);
    n += align_up(sizeof(NodeState) * (size_t)B * N, 256);
    n += align_up(sizeof(ShardAux) * (size_t)B * N, 256);
    n += align_up(sizeof(ShardPick) * (size_t)B, 256);
    return n;
}

static ShardLayout shard_layout(void* workspace, int B, int N) {
    char* base = static_cast<char*>(workspace) + sizeof(WorkspaceHeader);
    ShardLayout l;
    l.state = reinterpret_cast<NodeState*>(base);
    base += align_up(sizeof(NodeState) * (size_t)B * N, 256);
    l.aux = reinterpret_cast<ShardAux*>(base);
    base += align_up(sizeof(ShardAux) * (size_t)B * N, 256);
    l.pick = reinterpret_cast<ShardPick*>(base);
    return l;
}

// (p_u(x), q_u(x)) of every candidate node's token x under its parent u, where this rank owns x; zeros elsewhere
__global__ void verify_shard_gather_kernel(ProbRows rows, const int32_t* __restrict__ tokens,
                                           const int32_t* __restrict__ parent, const int32_t* __restrict__ level_start,
                                           int n_levels, const int32_t* __restrict__ gamma, int N, int Vs, int v0,
                                           double* __restrict__ pq) {
    const int b = blockIdx.x;
    const int n_act = active_nodes(gamma, level_start, n_levels, b, N);
    for (int c = threadIdx.x; c < N; c += blockDim.x) {
        double px = 0.0, qx = 0.0;
        const int u = parent[c];
        if (c < n_act && u >= 0 && u < N) {
            const int x = tokens[(size_t)b * N + c] - v0;
            if (x >= 0 && x < Vs) {
                px = (double)rows.p[((size_t)b * N + u) * Vs + x];
                qx = (double)rows.q[((size_t)b * N + u) * Vs + x];
            }
        }
        pq[((size_t)b * N + c) * 2] = px;
        pq[((size_t)b * N + c) * 2 + 1] = qx;
    }
}

// One round of the sibling loop for every node: takes the reduced mass of the pass issued last round (if any),
// tests the next sibling, and on a rejection sums this rank's part of the next residual mass into y.
__global__ void __launch_bounds__(kVerifyThreads)
verify_shard_round_kernel(ProbRows rows, const int32_t* __restrict__ parent, const int32_t* __restrict__ level_start,
                          int n_levels, const int32_t* __restrict__ gamma, const float* __restrict__ u_accept,
                          const double* __restrict__ pq, double* __restrict__ y, int round, int N, int Vs,
                          NodeState* __restrict__ state, ShardAux* __restrict__ aux) {
    __shared__ int s_first, s_cnt, s_pass;
    __shared__ double s_c;
    __shared__ VerifyScratch s_scratch;
    const int b = blockIdx.y, u = blockIdx.x, tid = threadIdx.x;
    const size_t i = (size_t)b * N + u;
    const int n_act = active_nodes(gamma, level_start, n_levels, b, N);
    if (u >= n_act) {
        if (tid == 0) y[i] = 0.0;
        return;
    }
    int first, cnt;
    find_children(parent, u, N, &s_first, &s_cnt, first, cnt);
    if (tid == 0) {
        NodeState st;
        ShardAux a;
        if (round == 0) {
            st.next_child = -1; st.top = -1; st.c = 0.0;
            a.pending = 0; a.c = 0.0; a.Y = 1.0;
            // in level order a kept prefix of the tree keeps either all children of a node or none
            a.stage = (cnt > 0 && first < n_act) ? 0 : -1;
        } else {
            st = state[i];
            a = aux[i];
        }
        int pass = 0;
        if (a.stage >= 0) {
            if (a.pending) {
                double Y = y[i];
                if (!(Y > 0.0)) { a.c = 0.0; Y = 1.0; }        // nothing left: back to the un-residualised row
                a.Y = Y;
                a.pending = 0;
                ++a.stage;
            }
            if (a.stage >= cnt) {                               // every sibling rejected: the walk stops here
                st.next_child = -1;
                st.c = a.c;
                a.stage = -1;
            } else {
                const int child = first + a.stage;
                const double px = pq[((size_t)b * N + child) * 2], qx = pq[((size_t)b * N + child) * 2 + 1];
                const double num = fmax(px - a.c * qx, 0.0);
                const double acc = qx > 0.0 ? fmin(1.0, num / (a.Y * qx)) : (num > 0.0 ? 1.0 : 0.0);
                if ((double)u_accept[(size_t)b * N + child] < acc) {
                    st.next_child = child;
                    a.stage = -1;
                } else {
                    a.c += a.Y;
                    a.pending = 1;
                    pass = 1;
                }
            }
        }
        state[i] = st;
        aux[i] = a;
        s_pass = pass;
        s_c = a.c;
    }
    __syncthreads();
    if (!s_pass) {
        if (tid == 0) y[i] = 0.0;
        return;
    }
    ProbDist d = rows.open(b, u, N, Vs, &s_scratch);
    d.set_c(s_c);
    const double part = dist_mass(d, &s_scratch);
    if (tid == 0) y[i] = part;
}

// Longest path (computed alike on every rank), then this rank's share of the stop distribution's mass and its
// last id with mass, written to row `rank` of the gather buffer (the other rows are zeroed for a sum-gather).
__global__ void __launch_bounds__(kVerifyThreads)
verify_shard_select_kernel(ProbRows rows, const int32_t* __restrict__ tokens, const NodeState* __restrict__ state,
                           int n_levels, int n_roots, int N, int Vs, int v0, int rank, int world, int B,
                           int32_t* __restrict__ accept_len, int32_t* __restrict__ out_tokens,
                           int32_t* __restrict__ out_nodes, int32_t* __restrict__ best_root,
                           double* __restrict__ mass, ShardPick* __restrict__ pick) {
    constexpr int E = ProbDist::E;
    __shared__ int s_len[MCSD_MAX_NODES];
    __shared__ int s_stop, s_slot;
    __shared__ VerifyScratch s_scratch;
    __shared__ CdfScratch s_cdf;
    const int b = blockIdx.x, tid = threadIdx.x;
    const NodeState* st = state + (size_t)b * N;
    select_path(st, tokens, b, n_levels, n_roots, N, accept_len, out_tokens, out_nodes, best_root, s_len, &s_stop, &s_slot);
    const int u = s_stop;
    ProbDist d = rows.open(b, u, N, Vs, &s_scratch);
    d.set_c(st[u].c);
    auto keep = [](int, float (&)[E]) {};
    cdf_range_sums_dist(d, keep, Vs, &s_cdf);
    if (tid == 0) {
        double total = 0.0;
        int last = -1;
        for (int w = 0; w < kVerifyWarps; ++w) { total += s_cdf.tot[w]; last = max(last, s_cdf.last[w]); }
        for (int r = 0; r < world; ++r) {
            mass[((size_t)r * B + b) * 2] = r == rank ? total : 0.0;
            mass[((size_t)r * B + b) * 2 + 1] = (r == rank && last >= 0) ? (double)(v0 + last + 1) : 0.0;
        }
        pick[b].stop = u;
        pick[b].slot = s_slot;
    }
}

// New token by inverse CDF in token-id order over the whole vocabulary: ranks are taken in order of their
// columns, the rank in whose columns the running sum passes u * total finishes the search locally.  Every rank
// writes out_tokens[b][slot]: the owner the token, the others -1 (a max over ranks then gives the token).
__global__ void __launch_bounds__(kVerifyThreads)
verify_shard_pick_kernel(ProbRows rows, const NodeState* __restrict__ state, const float* __restrict__ u_bonus,
                         int n_levels, int N, int Vs, int v0, int V_total, int rank, int world, int B,
                         const double* __restrict__ mass, const ShardPick* __restrict__ pick,
                         int32_t* __restrict__ out_tokens) {
    constexpr int E = ProbDist::E;
    __shared__ VerifyScratch s_scratch;
    __shared__ CdfScratch s_cdf;
    const int b = blockIdx.x, tid = threadIdx.x;
    const int u = pick[b].stop, slot = pick[b].slot;
    double total = 0.0;
    for (int r = 0; r < world; ++r) total += mass[((size_t)r * B + b) * 2];
    const double target = (double)u_bonus[(size_t)b * N + u] * total;
    double base = 0.0;
    int owner = -1;
    for (int r = 0; r < world; ++r) {
        const double m = mass[((size_t)r * B + b) * 2];
        if (base + m > target) { owner = r; break; }
        base += m;
    }
    int tok = -1;
    if (owner < 0) {                                            // nothing passes the target: last id with mass
        double last = 0.0;
        for (int r = 0; r < world; ++r) last = fmax(last, mass[((size_t)r * B + b) * 2 + 1]);
        tok = last > 0.0 ? (int)last - 1 : V_total - 1;
    } else if (owner == rank) {
        ProbDist d = rows.open(b, u, N, Vs, &s_scratch);
        d.set_c(state[(size_t)b * N + u].c);
        auto load = [&d](int idx, float (&r)[E]) { d.load(idx, r); };
        auto keep = [](int, float (&)[E]) {};
        cdf_range_sums_dist(d, keep, Vs, &s_cdf);
        double local_total;
        tok = v0 + cdf_locate<E>(load, target - base, true, Vs, &s_cdf, &local_total);
    }
    if (tid == 0) out_tokens[(size_t)b * (n_levels + 1) + slot] = tok;
}

static int check_shard_sizes(int B, int N, int Vs, int v0, int V_total) {
    if (B < 1 || N < 1 || Vs < 1 || N > MCSD_MAX_NODES || B > 65535) return MCSD_ERR_BAD_SHAPE;
    if (v0 < 0 || V_total < 1 || (long long)v0 + Vs > V_total) return MCSD_ERR_BAD_SHAPE;
    return MCSD_OK;
}

}  // namespace mcsd

extern "C" size_t mcsd_verify_shard_workspace_bytes(int B, int N) {
    if (B < 1 || N < 1) return 0;
    return mcsd::shard_workspace_bytes(B, N);
}

extern "C" int mcsd_verify_shard_gather(const float* p_shard, const float* q_shard, const int32_t* tokens,
                                        const int32_t* parent, const int32_t* level_start, int n_levels,
                                        const int32_t* gamma, int B, int N, int Vs, int v0, int V_total,
                                        double* pq_exchange, void* stream) {
    if (!p_shard || !q_shard || !tokens || !parent || !level_start || !pq_exchange) return MCSD_ERR_NULL;
    const int chk = mcsd::check_shard_sizes(B, N, Vs, v0, V_total);
    if (chk != MCSD_OK) return chk;
    if (n_levels < 1 || n_levels > N) return MCSD_ERR_BAD_SHAPE;
    const mcsd::ProbRows rows{p_shard, q_shard};
    mcsd::verify_shard_gather_kernel<<<B, 192, 0, static_cast<cudaStream_t>(stream)>>>(
        rows, tokens, parent, level_start, n_levels, gamma, N, Vs, v0, pq_exchange);
    MCSD_CUDA_CHECK(cudaGetLastError());
    mcsd::count_launches(1);
    return MCSD_OK;
}

extern "C" int mcsd_verify_shard_round(const float* p_shard, const float* q_shard, const int32_t* parent,
                                       const int32_t* level_start, int n_levels, const int32_t* gamma,
                                       const float* u_accept, const double* pq_exchange, double* y_exchange,
                                       int round, int B, int N, int Vs, void* workspace, size_t workspace_bytes,
                                       void* stream) {
    if (!p_shard || !q_shard || !parent || !level_start || !u_accept || !pq_exchange || !y_exchange || !workspace)
        return MCSD_ERR_NULL;
    const int chk = mcsd::check_shard_sizes(B, N, Vs, 0, Vs);
    if (chk != MCSD_OK) return chk;
    if (n_levels < 1 || n_levels > N || round < 0 || round > N) return MCSD_ERR_BAD_SHAPE;
    if (workspace_bytes < mcsd::shard_workspace_bytes(B, N)) return MCSD_ERR_WORKSPACE_TOO_SMALL;
    const mcsd::ShardLayout l = mcsd::shard_layout(workspace, B, N);
    const mcsd::ProbRows rows{p_shard, q_shard};
    mcsd::verify_shard_round_kernel<<<dim3(N, B), mcsd::kVerifyThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        rows, parent, level_start, n_levels, gamma, u_accept, pq_exchange, y_exchange, round, N, Vs, l.state, l.aux);
    MCSD_CUDA_CHECK(cudaGetLastError());
    mcsd::count_launches(1);
    return MCSD_OK;
}

extern "C" int mcsd_verify_shard_select(const float* p_shard, const float* q_shard, const int32_t* tokens,
                                        int n_levels, int n_roots, int B, int N, int Vs, int v0, int V_total,
                                        int rank, int world, int32_t* accept_len, int32_t* out_tokens,
                                        int32_t* out_nodes, int32_t* best_root, double* mass_exchange,
                                        void* workspace, size_t workspace_bytes, void* stream) {
    if (!p_shard || !q_shard || !tokens || !accept_len || !out_tokens || !out_nodes || !best_root || !mass_exchange ||
        !workspace)
        return MCSD_ERR_NULL;
    const int chk = mcsd::check_shard_sizes(B, N, Vs, v0, V_total);
    if (chk != MCSD_OK) return chk;
    if (n_levels < 1 || n_levels > N || n_roots < 1 || n_roots > N) return MCSD_ERR_BAD_SHAPE;
    if (world < 1 || world > 1024 || rank < 0 || rank >= world) return MCSD_ERR_BAD_SHAPE;
    if (workspace_bytes < mcsd::shard_workspace_bytes(B, N)) return MCSD_ERR_WORKSPACE_TOO_SMALL;
    const mcsd::ShardLayout l = mcsd::shard_layout(workspace, B, N);
    const mcsd::ProbRows rows{p_shard, q_shard};
    mcsd::verify_shard_select_kernel<<<B, mcsd::kVerifyThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        rows, tokens, l.state, n_levels, n_roots, N, Vs, v0, rank, world, B, accept_len, out_tokens, out_nodes,
        best_root, mass_exchange, l.pick);
    MCSD_CUDA_CHECK(cudaGetLastError());
    mcsd::count_launches(1);
    return MCSD_OK;
}

extern "C" int mcsd_verify_shard_pick(const float* p_shard, const float* q_shard, const float* u_bonus, int n_levels,
                                      int B, int N, int Vs, int v0, int V_total, int rank, int world,
                                      const double* mass_exchange, int32_t* out_tokens, const void* workspace,
                                      size_t workspace_bytes, void* stream) {
    if (!p_shard || !q_shard || !u_bonus || !mass_exchange || !out_tokens || !workspace) return MCSD_ERR_NULL;
    const int chk = mcsd::check_shard_sizes(B, N, Vs, v0, V_total);
    if (chk != MCSD_OK) return chk;
    if (n_levels < 1 || n_levels > N) return MCSD_ERR_BAD_SHAPE;
    if (world < 1 || world > 1024 || rank < 0 || rank >= world) return MCSD_ERR_BAD_SHAPE;
    if (workspace_bytes < mcsd::shard_workspace_bytes(B, N)) return MCSD_ERR_WORKSPACE_TOO_SMALL;
    const mcsd::ShardLayout l = mcsd::shard_layout(const_cast<void*>(workspace), B, N);
    const mcsd::ProbRows rows{p_shard, q_shard};
    mcsd::verify_shard_pick_kernel<<<B, mcsd::kVerifyThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        rows, l.state, u_bonus, n_levels, N, Vs, v0, V_total, rank, world, B, mass_exchange, l.pick, out_tokens);
    MCSD_CUDA_CHECK(cudaGetLastError());
    mcsd::count_launches(1);
    return MCSD_OK;
}
