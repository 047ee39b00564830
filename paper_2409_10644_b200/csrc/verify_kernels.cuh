// Multi-candidate accept/reject over a token tree (Fig. 1 steps 4-6 of the paper; Section 3.1 for several
// target-initialised roots): the kernels, written once for every way the two next-token distributions can
// be given (probability rows, or logit rows with a temperature).
//
// The walk of one root visits a node, tries its children in order and either moves to the first accepted
// child or stops.  Uniforms are indexed by node, so what happens at a node does not depend on how the walk
// got there.  That splits the work in two phases of one launch:
//
//   node phase            one thread block per (sequence, node): decides which child, if any, is accepted
//                         at that node.  After m rejections the target-side distribution is
//                         max(p - c_m q, 0) / Y_m with c_0 = 0, Y_0 = 1, c_{m+1} = c_m + Y_m and
//                         Y_m = sum_v max(p_v - c_m q_v, 0): iterating norm(max(pt - q, 0)) never needs a
//                         vocabulary-sized write, only one reduction over the two rows per rejection.
//   select phase          the block of a sequence that finishes its node last (a ticket per sequence in the
//                         workspace; nothing waits): follows next_child from every root, keeps the longest
//                         path (ties: lowest root), then draws the new token at its stop node by inverse CDF
//                         in token-id order and, on request, lists the most probable ids.
//
// A "Rows" type hands out, for one (sequence, node), a "Dist": the pair of rows seen as the unnormalised
// distribution  dist_v = max(p_v - c q_v, 0)  for a settable c, read E ids at a time with 128-bit loads
// when the row allows.  Reductions run in a fixed order, fp32 per lane and fp64 across warps.
#pragma once

#include <cuda_bf16.h>

#include "common.cuh"

namespace mcsd {

#ifndef MCSD_VERIFY_THREADS
#define MCSD_VERIFY_THREADS 512
#endif
constexpr int kVerifyThreads = MCSD_VERIFY_THREADS;
constexpr int kVerifyWarps = kVerifyThreads / 32;

struct NodeState {
    int32_t next_child;   // accepted child, or -1 if the walk stops here
    int32_t top;          // greedy verification: id of the largest target logit of this node
    double c;             // stop distribution is max(p - c q, 0); c = 0 means the row p itself
};

// Workspace layout of the verify calls: header, B * N node states, then one ticket per sequence (arrivals of the
// sequence's node blocks; zero between launches).
inline size_t verify_tickets_offset(int B, int N) {
    return align_up(sizeof(WorkspaceHeader) + sizeof(NodeState) * (size_t)B * N, 256);
}

// block-wide scratch of the row passes
struct VerifyScratch {
    double warp_sum[kVerifyWarps];
    float stat_m[2][kVerifyWarps];
    float stat_s[2][kVerifyWarps];
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <int E> __device__ __forceinline__ float tree_sum(const float (&r)[E]) {
    if constexpr (E == 4) {
        return (r[0] + r[1]) + (r[2] + r[3]);
    } else {
        static_assert(E == 8, "4 or 8 ids per load");
        return ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
    }
}

// ------------------------------------------------------------------------------------------------------
// probability rows: p, q are fp32 distributions
// ------------------------------------------------------------------------------------------------------
struct ProbDist {
    static constexpr int E = 4;
    const float* p;
    const float* q;
    int V;
    bool vec;
    float c;

    __device__ __forceinline__ void set_c(double c_) { c = (float)c_; }
    __device__ __forceinline__ double p_of(int x) const { return (double)p[x]; }
    __device__ __forceinline__ double q_of(int x) const { return (double)q[x]; }

    __device__ __forceinline__ static void load_row(const float* __restrict__ row, int idx, int V, bool vec, float (&r)[4]) {
        if (vec) {
            const float4 t = __ldg(reinterpret_cast<const float4*>(row + idx));
            r[0] = t.x; r[1] = t.y; r[2] = t.z; r[3] = t.w;
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) r[i] = idx + i < V ? __ldg(row + idx + i) : 0.f;
        }
    }
    __device__ __forceinline__ void load(int idx, float (&r)[4]) const {
        load_row(p, idx, V, vec, r);
        if (c != 0.f) {
            float b[4];
            load_row(q, idx, V, vec, b);
#pragma unroll
            for (int i = 0; i < 4; ++i) r[i] = fmaxf(fmaf(-c, b[i], r[i]), 0.f);
        }
    }
    // The same values in two steps, for row passes that issue the loads of several steps before using any of
    // them (only for rows that allow 128-bit loads): PLAIN = the row p itself (c == 0), no draft row needed.
    __device__ __forceinline__ bool plain() const { return c == 0.f; }
    template <bool PLAIN> __device__ __forceinline__ void fetch(int idx, float (&a)[4], float (&b)[4]) const {
        const float4 t = __ldg(reinterpret_cast<const float4*>(p + idx));
        a[0] = t.x; a[1] = t.y; a[2] = t.z; a[3] = t.w;
        if constexpr (!PLAIN) {
            const float4 s = __ldg(reinterpret_cast<const float4*>(q + idx));
            b[0] = s.x; b[1] = s.y; b[2] = s.z; b[3] = s.w;
        }
    }
    template <bool PLAIN> __device__ __forceinline__ void finish(const float (&a)[4], const float (&b)[4], float (&r)[4]) const {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if constexpr (PLAIN) r[i] = a[i];
            else r[i] = fmaxf(fmaf(-c, b[i], a[i]), 0.f);
        }
    }
};

struct ProbRows {
    using Dist = ProbDist;
    const float* p;
    const float* q;
    __device__ __forceinline__ Dist open(int b, int u, int N, int V, VerifyScratch*) const {
        Dist d;
        d.p = p + ((size_t)b * N + u) * V;
        d.q = q + ((size_t)b * N + u) * V;
        d.V = V;
        d.vec = (V % 4 == 0) && ((reinterpret_cast<uintptr_t>(d.p) | reinterpret_cast<uintptr_t>(d.q)) % 16 == 0);
        d.c = 0.f;
        return d;
    }
};

// ------------------------------------------------------------------------------------------------------
// logit rows with a temperature T > 0 (Fig. 1 step 4): p_v = exp(zt_v / T) / sum_w exp(zt_w / T), q likewise
// from the draft logits.  Opening a node costs one pass over both rows (running maximum and sum per thread,
// merged across the block); afterwards p_v and q_v are formed on the fly, never stored.
// ------------------------------------------------------------------------------------------------------
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <typename T> struct LogitLoad;
template <> struct LogitLoad<float> {
    static constexpr int E = 4;
    __device__ __forceinline__ static void load(const float* __restrict__ row, int idx, int V, bool vec, float (&r)[4]) {
        if (vec) {
            const float4 t = __ldg(reinterpret_cast<const float4*>(row + idx));
            r[0] = t.x; r[1] = t.y; r[2] = t.z; r[3] = t.w;
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) r[i] = idx + i < V ? __ldg(row + idx + i) : -INFINITY;
        }
    }
    __device__ __forceinline__ static void load_vec(const float* __restrict__ row, int idx, float (&r)[4]) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(row + idx));
        r[0] = t.x; r[1] = t.y; r[2] = t.z; r[3] = t.w;
    }
    __device__ __forceinline__ static float one(const float* row, int x) { return row[x]; }
};
template <> struct LogitLoad<__nv_bfloat16> {
    static constexpr int E = 8;
    __device__ __forceinline__ static void load(const __nv_bfloat16* __restrict__ row, int idx, int V, bool vec, float (&r)[8]) {
        if (vec) {
            const uint4 t = __ldg(reinterpret_cast<const uint4*>(row + idx));
            const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {          // a bf16 is the upper half of the fp32 with the same value
                r[2 * i] = __uint_as_float(w[i] << 16);
                r[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) r[i] = idx + i < V ? __bfloat162float(row[idx + i]) : -INFINITY;
        }
    }
    __device__ __forceinline__ static void load_vec(const __nv_bfloat16* __restrict__ row, int idx, float (&r)[8]) {
        const uint4 t = __ldg(reinterpret_cast<const uint4*>(row + idx));
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            r[2 * i] = __uint_as_float(w[i] << 16);
            r[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    __device__ __forceinline__ static float one(const __nv_bfloat16* row, int x) { return __bfloat162float(row[x]); }
};

// (m1, s1) + (m2, s2) for sums of exp2((z - m) k)
__device__ __forceinline__ void merge_stat(float& m, float& s, float m2, float s2, float k) {
    const float mn = fmaxf(m, m2);
    if (mn == -INFINITY) return;                    // neither side has seen a finite logit
    s = s * ex2f((m - mn) * k) + s2 * ex2f((m2 - mn) * k);
    m = mn;
}

template <typename T> struct LogitDist {
    static constexpr int E = LogitLoad<T>::E;
    const T* zt;
    const T* zd;
    int V;
    bool vec;
    float k;              // log2(e) / T
    float mt, md;         // row maxima
    double Zp, Zq;        // sum_v exp2((z_v - m) k)
    float ip, cq;         // 1 / Zp and c / Zq

    __device__ __forceinline__ void set_c(double c) { cq = (float)(c / Zq); }
    __device__ __forceinline__ double p_of(int x) const {
        return exp2(((double)LogitLoad<T>::one(zt, x) - (double)mt) * (double)k) / Zp;
    }
    __device__ __forceinline__ double q_of(int x) const {
        return exp2(((double)LogitLoad<T>::one(zd, x) - (double)md) * (double)k) / Zq;
    }
    __device__ __forceinline__ void load(int idx, float (&r)[E]) const {
        LogitLoad<T>::load(zt, idx, V, vec, r);
#pragma unroll
        for (int i = 0; i < E; ++i) r[i] = ex2f((r[i] - mt) * k) * ip;
        if (cq != 0.f) {
            float b[E];
            LogitLoad<T>::load(zd, idx, V, vec, b);
#pragma unroll
            for (int i = 0; i < E; ++i) r[i] = fmaxf(fmaf(-cq, ex2f((b[i] - md) * k), r[i]), 0.f);
        }
    }

    __device__ __forceinline__ bool plain() const { return cq == 0.f; }
    template <bool PLAIN> __device__ __forceinline__ void fetch(int idx, float (&a)[E], float (&b)[E]) const {
        LogitLoad<T>::load_vec(zt, idx, a);
        if constexpr (!PLAIN) LogitLoad<T>::load_vec(zd, idx, b);
    }
    template <bool PLAIN> __device__ __forceinline__ void finish(const float (&a)[E], const float (&b)[E], float (&r)[E]) const {
#pragma unroll
        for (int i = 0; i < E; ++i) {
            r[i] = ex2f((a[i] - mt) * k) * ip;
            if constexpr (!PLAIN) r[i] = fmaxf(fmaf(-cq, ex2f((b[i] - md) * k), r[i]), 0.f);
        }
    }

    // maxima and normalisers of both rows; every thread of the block must call it
    __device__ void stats(VerifyScratch* sc) {
        float m[2] = {-INFINITY, -INFINITY}, s[2] = {0.f, 0.f};
        const float kk = k;
        auto fold = [&m, &s, kk](int row, const float (&a)[E]) {
            float vm = a[0];
#pragma unroll
            for (int i = 1; i < E; ++i) vm = fmaxf(vm, a[i]);
            if (vm == -INFINITY) return;
            if (vm > m[row]) { s[row] *= ex2f((m[row] - vm) * kk); m[row] = vm; }
            float e[E];
#pragma unroll
            for (int i = 0; i < E; ++i) e[i] = ex2f((a[i] - m[row]) * kk);
            s[row] += tree_sum<E>(e);
        };
        constexpr int kStep = kVerifyThreads * E;
        constexpr int kBatch = E == 8 ? 2 : 4;  // steps whose loads are issued before the first one is folded in
        int idx = threadIdx.x * E;
        if (vec) {
            for (; idx + (kBatch - 1) * kStep < V; idx += kBatch * kStep) {
                float at[kBatch][E], ad[kBatch][E];
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    LogitLoad<T>::load_vec(zt, idx + j * kStep, at[j]);
                    LogitLoad<T>::load_vec(zd, idx + j * kStep, ad[j]);
                }
#pragma unroll
                for (int j = 0; j < kBatch; ++j) { fold(0, at[j]); fold(1, ad[j]); }
            }
        }
        for (; idx < V; idx += kStep) {
#pragma unroll
            for (int row = 0; row < 2; ++row) {
                float a[E];
                LogitLoad<T>::load(row == 0 ? zt : zd, idx, V, vec, a);
                fold(row, a);
            }
        }
#pragma unroll
        for (int row = 0; row < 2; ++row) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float m2 = __shfl_xor_sync(0xffffffffu, m[row], o);
                const float s2 = __shfl_xor_sync(0xffffffffu, s[row], o);
                merge_stat(m[row], s[row], m2, s2, k);
            }
        }
        __syncthreads();                            // the scratch may still be read from a previous pass
        if ((threadIdx.x & 31) == 0) {
            sc->stat_m[0][threadIdx.x >> 5] = m[0]; sc->stat_s[0][threadIdx.x >> 5] = s[0];
            sc->stat_m[1][threadIdx.x >> 5] = m[1]; sc->stat_s[1][threadIdx.x >> 5] = s[1];
        }
        __syncthreads();
        double Z[2];
        float M[2];
#pragma unroll
        for (int row = 0; row < 2; ++row) {
            float mm = -INFINITY;
            for (int w = 0; w < kVerifyWarps; ++w) mm = fmaxf(mm, sc->stat_m[row][w]);
            double z = 0.0;
            for (int w = 0; w < kVerifyWarps; ++w) {
                const float mw = sc->stat_m[row][w];
                if (mw != -INFINITY) z += (double)sc->stat_s[row][w] * (double)ex2f((mw - mm) * k);
            }
            M[row] = mm; Z[row] = z;
        }
        mt = M[0]; md = M[1];
        Zp = Z[0] > 0.0 ? Z[0] : 1.0;
        Zq = Z[1] > 0.0 ? Z[1] : 1.0;
        ip = (float)(1.0 / Zp);
        cq = 0.f;
    }
};

template <typename T> struct LogitRows {
    using Dist = LogitDist<T>;
    const T* zt;
    const T* zd;
    float k;
    __device__ __forceinline__ Dist open(int b, int u, int N, int V, VerifyScratch* sc) const {
        Dist d;
        d.zt = zt + ((size_t)b * N + u) * V;
        d.zd = zd + ((size_t)b * N + u) * V;
        d.V = V;
        d.vec = (V % Dist::E == 0) && ((reinterpret_cast<uintptr_t>(d.zt) | reinterpret_cast<uintptr_t>(d.zd)) % 16 == 0);
        d.k = k;
        d.stats(sc);
        return d;
    }
};

// ------------------------------------------------------------------------------------------------------
// row passes shared by both kernels
// ------------------------------------------------------------------------------------------------------

// Row passes are latency-bound for a single block (one step = one dependent trip to memory), so they run
// kRowBatch steps at a time: all loads of the batch are issued before the first value is used.  The additions
// keep the order of the plain loop, so the sums are the same bit for bit.
constexpr int kRowBatch = 4;
// two-row passes over 8-id loads keep two steps in flight: four would cost the node kernel half its resident blocks

// this thread's part of sum_v dist_v: ids first, first + step, ... below end
template <bool PLAIN, typename Dist>
__device__ __forceinline__ float strided_sum(const Dist& d, int first, int step, int end) {
    constexpr int E = Dist::E;
    constexpr int NB = E == 8 ? 2 : kRowBatch;
    float acc = 0.f;
    int idx = first;
    for (; idx + (NB - 1) * step < end; idx += NB * step) {
        float a[NB][E], b[NB][E];
#pragma unroll
        for (int j = 0; j < NB; ++j) d.template fetch<PLAIN>(idx + j * step, a[j], b[j]);
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            float r[E];
            d.template finish<PLAIN>(a[j], b[j], r);
            acc += tree_sum<E>(r);
        }
    }
    for (; idx < end; idx += step) {
        float r[E];
        d.load(idx, r);
        acc += tree_sum<E>(r);
    }
    return acc;
}

// sum_v dist_v over one row, same value in every thread of the block
template <typename Dist> __device__ double dist_mass(const Dist& d, VerifyScratch* sc) {
    constexpr int E = Dist::E;
    float acc = 0.f;
    if (d.vec) {
        acc = d.plain() ? strided_sum<true>(d, threadIdx.x * E, kVerifyThreads * E, d.V)
                        : strided_sum<false>(d, threadIdx.x * E, kVerifyThreads * E, d.V);
    } else {
        for (int idx = threadIdx.x * E; idx < d.V; idx += kVerifyThreads * E) {
            float r[E];
            d.load(idx, r);
            acc += tree_sum<E>(r);
        }
    }
    acc = warp_sum(acc);
    __syncthreads();                       // the scratch may still be read from a previous pass
    if ((threadIdx.x & 31) == 0) sc->warp_sum[threadIdx.x >> 5] = (double)acc;
    __syncthreads();
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < kVerifyWarps; ++w) tot += sc->warp_sum[w];
    return tot;
}

__device__ __forceinline__ int active_nodes(const int32_t* gamma, const int32_t* level_start, int n_levels, int b, int N) {
    if (gamma == nullptr) return N;
    int g = gamma[b];
    g = g < 0 ? 0 : (g > n_levels - 1 ? n_levels - 1 : g);
    return min(level_start[g + 1], N);
}

// children of node u: first id and count, same values in every thread of the block
__device__ __forceinline__ void find_children(const int32_t* __restrict__ parent, int u, int N, int* s_first, int* s_cnt,
                                              int& first, int& cnt) {
    if (threadIdx.x == 0) { *s_first = N; *s_cnt = 0; }
    __syncthreads();
    for (int c = threadIdx.x; c < N; c += blockDim.x)
        if (parent[c] == u) { atomicMin(s_first, c); atomicAdd(s_cnt, 1); }
    __syncthreads();
    first = *s_first;
    cnt = *s_cnt;
}

// (value, id) order used for the list of most probable ids: larger value first, ties to the smaller id
__device__ __forceinline__ bool better(float va, int ia, float vb, int ib) {
    return va > vb || (va == vb && ia < ib);
}

// Follows next_child from every root, keeps the longest path (ties: lowest root) and writes accept_len,
// best_root, out_nodes and all of out_tokens but the new token.  Returns the stop node and the slot of the
// new token through shared memory (and the stop node's residual coefficient, if asked for); ends with a block
// barrier.  The sequence's node states and tokens are brought into shared memory with one trip to memory and the
// walks run there: followed through global memory, every step of every walk was a dependent trip of its own.
__device__ __forceinline__ void select_path(const NodeState* __restrict__ st, const int32_t* __restrict__ tokens, int b,
                                            int n_levels, int n_roots, int N, int32_t* __restrict__ accept_len,
                                            int32_t* __restrict__ out_tokens, int32_t* __restrict__ out_nodes,
                                            int32_t* __restrict__ best_root, int* s_len, int* s_stop, int* s_slot,
                                            double* s_c_stop = nullptr, const float* __restrict__ u_bonus = nullptr,
                                            float* s_u_stop = nullptr) {
    __shared__ int s_next[MCSD_MAX_NODES];
    __shared__ int s_tok[MCSD_MAX_NODES];
    __shared__ double s_c[MCSD_MAX_NODES];
    __shared__ float s_ub[MCSD_MAX_NODES];
    const int tid = threadIdx.x;
    for (int i = tid; i < N; i += blockDim.x) {
        s_next[i] = __ldcg(&st[i].next_child);
        s_c[i] = __ldcg(&st[i].c);
        s_tok[i] = tokens[(size_t)b * N + i];
        if (u_bonus) s_ub[i] = u_bonus[(size_t)b * N + i];
    }
    __syncthreads();
    if (tid < n_roots) {
        int u = tid, len = 0;
        for (int step = 0; step < n_levels; ++step) {
            const int nc = s_next[u];
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
        if (n_roots > 1) ot[slot++] = s_tok[best];
        int u = best;
        for (int i = 0; i < s_len[best]; ++i) {
            u = s_next[u];
            on[i] = u;
            ot[slot++] = s_tok[u];
        }
        accept_len[b] = s_len[best];
        best_root[b] = best;
        *s_stop = u;
        *s_slot = slot;
        if (s_c_stop) *s_c_stop = s_c[u];
        if (s_u_stop && u_bonus) *s_u_stop = s_ub[u];
    }
    __syncthreads();
}

// The R ids with the largest value(id) (ties to the smaller id), by R selection passes over the row.
// `load(idx, r)` fills E values starting at id idx; ids >= V are ignored.
template <int E, typename Load>
__device__ void top_ids(const Load& load, int V, int R, int32_t* __restrict__ dst, float* s_bv, int* s_bi) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float pv = __int_as_float(0x7f800000);   // previous pick: +inf, id -1
    int pi = -1;
    for (int r = 0; r < R; ++r) {
        float bv = 0.f;
        int bi = -1;
        for (int idx = tid * E; idx < V; idx += kVerifyThreads * E) {
            float ev[E];
            load(idx, ev);
#pragma unroll
            for (int k = 0; k < E; ++k) {
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
        if (tid == 0) dst[r] = bi;
        pv = bv; pi = bi;
        if (bi < 0) {                       // fewer than R ids in the vocabulary
            for (int rr = r + 1 + tid; rr < R; rr += kVerifyThreads) dst[rr] = -1;
            break;
        }
    }
}

// Inverse CDF in token-id order over the unnormalised distribution `load` hands out E ids at a time: the smallest
// id t whose running sum exceeds u * total; if rounding lets nothing exceed it, the last id with mass (V - 1 if
// there is none).  Every thread of the block must call it; all get the id, and *total_out the total mass.
// pass 1: every warp sums one contiguous range of ids; pass 2: one warp locates the crossing, starting in the
// range where the running sum passes u * total.
struct CdfScratch {
    double tot[kVerifyWarps];
    int last[kVerifyWarps];
    float ctot[kVerifyWarps];     // locate: totals of the chunks scanned side by side
    int cand[kVerifyWarps];       // locate: id found in each of them, or -1
};
// pass 1: per-warp range sums and last id with mass, left in the scratch; ends with a block barrier
template <int E, typename Load>
__device__ void cdf_range_sums(const Load& load, int V, CdfScratch* sc) {
    constexpr int kStride = 32 * E;             // ids one warp covers per step
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int span = ((V + kVerifyWarps - 1) / kVerifyWarps + kStride - 1) / kStride * kStride;
    __syncthreads();                            // the scratch may still be read from a previous call
    {
        const int lo = warp * span, hi = min(V, lo + span);
        float acc = 0.f;
        int last = -1;
        for (int idx = lo + lane * E; idx < hi; idx += kStride) {
            float r[E];
            load(idx, r);
            acc += tree_sum<E>(r);
#pragma unroll
            for (int i = 0; i < E; ++i)
                if (r[i] > 0.f) last = idx + i;
        }
        acc = warp_sum(acc);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
        if (lane == 0) { sc->tot[warp] = (double)acc; sc->last[warp] = last; }
    }
    __syncthreads();
}

// pass 1 for a Dist whose values `post(idx, r)` may still edit (e.g. to drop ids): batched loads when the rows
// allow 128-bit loads (see strided_sum), the plain pass otherwise.  Same sums as cdf_range_sums bit for bit.
template <bool PLAIN, typename Dist, typename Post>
__device__ __forceinline__ void range_sum_batched(const Dist& d, const Post& post, int first, int step, int end,
                                                  float& acc, int& last) {
    constexpr int E = Dist::E;
    constexpr int NB = E == 8 ? 2 : kRowBatch;
    int idx = first;
    for (; idx + (NB - 1) * step < end; idx += NB * step) {
        float a[NB][E], b[NB][E];
#pragma unroll
        for (int j = 0; j < NB; ++j) d.template fetch<PLAIN>(idx + j * step, a[j], b[j]);
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            float r[E];
            d.template finish<PLAIN>(a[j], b[j], r);
            post(idx + j * step, r);
            acc += tree_sum<E>(r);
#pragma unroll
            for (int i = 0; i < E; ++i)
                if (r[i] > 0.f) last = idx + j * step + i;
        }
    }
    for (; idx < end; idx += step) {
        float r[E];
        d.load(idx, r);
        post(idx, r);
        acc += tree_sum<E>(r);
#pragma unroll
        for (int i = 0; i < E; ++i)
            if (r[i] > 0.f) last = idx + i;
    }
}

template <typename Dist, typename Post>
__device__ void cdf_range_sums_dist(const Dist& d, const Post& post, int V, CdfScratch* sc) {
    constexpr int E = Dist::E;
    if (!d.vec) {
        auto load = [&d, &post](int idx, float (&r)[E]) { d.load(idx, r); post(idx, r); };
        cdf_range_sums<E>(load, V, sc);
        return;
    }
    constexpr int kStride = 32 * E;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int span = ((V + kVerifyWarps - 1) / kVerifyWarps + kStride - 1) / kStride * kStride;
    __syncthreads();                            // the scratch may still be read from a previous call
    {
        const int lo = warp * span, hi = min(V, lo + span);
        float acc = 0.f;
        int last = -1;
        if (d.plain()) range_sum_batched<true>(d, post, lo + lane * E, kStride, hi, acc, last);
        else range_sum_batched<false>(d, post, lo + lane * E, kStride, hi, acc, last);
        acc = warp_sum(acc);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
        if (lane == 0) { sc->tot[warp] = (double)acc; sc->last[warp] = last; }
    }
    __syncthreads();
}

// pass 2, after cdf_range_sums: the smallest id whose running sum exceeds the target, which is t itself when
// `absolute` and t * (total mass) otherwise; the last id with mass (V - 1 if there is none) if nothing exceeds it.
// Every thread of the block must call it; all get the id, and *total_out the total mass.
template <int E, typename Load>
__device__ int cdf_locate(const Load& load, double t, bool absolute, int V, CdfScratch* sc, double* total_out) {
    constexpr int kStride = 32 * E;             // ids of one chunk: what a warp covers in one step
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int span = ((V + kVerifyWarps - 1) / kVerifyWarps + kStride - 1) / kStride * kStride;
    // every thread repeats the few additions over the range sums, so all agree without another barrier
    double total = 0.0;
    int last_pos = -1;
    for (int w = 0; w < kVerifyWarps; ++w) { total += sc->tot[w]; last_pos = max(last_pos, sc->last[w]); }
    const double target = absolute ? t : t * total;
    double base = 0.0;
    int w0 = 0;
    while (w0 < kVerifyWarps && !(base + sc->tot[w0] > target)) { base += sc->tot[w0]; ++w0; }
    // The running sum is carried chunk by chunk in id order, as a single warp walking the range would do, but
    // the chunks of a range are loaded and scanned by all warps at once: warp j takes chunk j, the chunk totals
    // are then added up in order, and the lowest chunk in which the sum passes the target gives the id.
    int found = -1;
    for (int w = w0; w < kVerifyWarps && found < 0; ++w) {
        const int lo = w * span, hi = min(V, lo + span);
        for (int c0 = lo; c0 < hi && found < 0; c0 += kVerifyWarps * kStride) {
            const int idx = c0 + warp * kStride + lane * E;
            float r[E];
#pragma unroll
            for (int i = 0; i < E; ++i) r[i] = 0.f;
            if (idx < hi) load(idx, r);
            const float ls = tree_sum<E>(r);
            float incl = ls;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float t2 = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t2;
            }
            if (lane == 31) sc->ctot[warp] = incl;
            __syncthreads();
            double mine = base, all = base;
            for (int k = 0; k < kVerifyWarps; ++k) {
                if (k == warp) mine = all;
                all += (double)sc->ctot[k];
            }
            const bool hit = (mine + (double)incl > target) && idx < hi;
            const unsigned ballot = __ballot_sync(0xffffffffu, hit);
            int tok = -1;
            if (ballot != 0u) {
                const int L = __ffs(ballot) - 1;
                if (lane == L) {
                    const double ex = mine + (double)(incl - ls);
                    float part = 0.f;
                    bool done = false;
                    tok = idx + E - 1;
#pragma unroll
                    for (int i = 0; i < E - 1; ++i) {        // smallest i whose running sum passes the target
                        part += r[i];
                        if (!done && ex + (double)part > target) { tok = idx + i; done = true; }
                    }
                    if (tok >= V) tok = V - 1;
                }
                tok = __shfl_sync(0xffffffffu, tok, L);
            }
            if (lane == 0) sc->cand[warp] = tok;
            __syncthreads();
            for (int k = 0; k < kVerifyWarps && found < 0; ++k) found = sc->cand[k];
            base = all;
            __syncthreads();                        // the chunk scratch is rewritten in the next step
        }
    }
    if (found < 0) found = last_pos >= 0 ? last_pos : V - 1;
    *total_out = total;
    return found;
}

template <int E, typename Load>
__device__ int block_inverse_cdf(const Load& load, float u, int V, CdfScratch* sc, double* total_out) {
    cdf_range_sums<E>(load, V, sc);
    return cdf_locate<E>(load, (double)u, false, V, sc, total_out);
}

// Select phase of one sequence, run by all threads of one block: the walk from every root, the longest path, the new
// token by inverse CDF at its stop node and, on request, the R most probable ids of the same distribution.
template <typename Rows>
__device__ void select_and_draw(const Rows& rows, const int32_t* __restrict__ tokens, const NodeState* st, int b, int n_levels,
                                int n_roots, const float* __restrict__ u_bonus, int N, int V, int32_t* __restrict__ accept_len,
                                int32_t* __restrict__ out_tokens, int32_t* __restrict__ out_nodes,
                                int32_t* __restrict__ best_root, int32_t* __restrict__ next_roots, int R,
                                VerifyScratch* s_scratch) {
    using Dist = typename Rows::Dist;
    constexpr int E = Dist::E;
    __shared__ int s_len[MCSD_MAX_NODES];
    __shared__ int s_stop, s_slot;
    __shared__ double s_c_stop;
    __shared__ float s_u_stop;
    __shared__ CdfScratch s_cdf;
    __shared__ float s_bv[kVerifyWarps];
    __shared__ int s_bi[kVerifyWarps];
    const int tid = threadIdx.x;

    select_path(st, tokens, b, n_levels, n_roots, N, accept_len, out_tokens, out_nodes, best_root, s_len, &s_stop, &s_slot,
                &s_c_stop, u_bonus, &s_u_stop);
    const int u = s_stop;
    Dist d = rows.open(b, u, N, V, s_scratch);
    d.set_c(s_c_stop);

    // ---- new token: inverse CDF over dist_v = max(p_v - c q_v, 0) in token-id order ----
    auto load = [&d](int idx, float (&r)[E]) { d.load(idx, r); };
    auto keep = [](int, float (&)[E]) {};
    double total;
    cdf_range_sums_dist(d, keep, V, &s_cdf);
    const int found = cdf_locate<E>(load, (double)s_u_stop, false, V, &s_cdf, &total);
    if (tid == 0) out_tokens[(size_t)b * (n_levels + 1) + s_slot] = found;

    // ---- optional: the R most probable ids of the same distribution ----
    if (next_roots != nullptr && R > 0) top_ids<E>(load, V, R, next_roots + (size_t)b * R, s_bv, s_bi);
}

template <typename Rows>
__global__ void __launch_bounds__(kVerifyThreads)
verify_tree_kernel(Rows rows, const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                   const int32_t* __restrict__ level_start, int n_levels, int n_roots, const int32_t* __restrict__ gamma,
                   const float* __restrict__ u_accept, const float* __restrict__ u_bonus, int N, int V,
                   NodeState* state, int* tickets, int32_t* __restrict__ accept_len, int32_t* __restrict__ out_tokens,
                   int32_t* __restrict__ out_nodes, int32_t* __restrict__ best_root, int32_t* __restrict__ next_roots, int R) {
    __shared__ int s_first, s_cnt, s_accept, s_last;
    __shared__ VerifyScratch s_scratch;
    __shared__ double s_px[MCSD_MAX_NODES], s_qx[MCSD_MAX_NODES];
    __shared__ float s_ua[MCSD_MAX_NODES];
    // Blocks are handed out in the order of their linear index; taking the node from its upper part starts all
    // sequences' nodes level by level, so the nodes with the most siblings to try run first and the leaves,
    // which have nothing to do, last.
    const int lin = blockIdx.y * gridDim.x + blockIdx.x;
    const int b = lin % (int)gridDim.y, u = lin / (int)gridDim.y, tid = threadIdx.x;
    const int n_act = active_nodes(gamma, level_start, n_levels, b, N);
    if (u >= n_act) return;                    // first: a sliced forest launches many blocks that have nothing to do
    // the sequence's tokens travel together with the parent array: one trip to memory instead of two in a row
    __shared__ int s_tok[MCSD_MAX_NODES];
    for (int i = tid; i < N; i += kVerifyThreads) s_tok[i] = tokens[(size_t)b * N + i];
    int first, cnt;
    find_children(parent, u, N, &s_first, &s_cnt, first, cnt);

    NodeState st;
    st.next_child = -1; st.top = -1; st.c = 0.0;
    // in level order a kept prefix of the tree keeps either all children of a node or none
    if (cnt > 0 && first < n_act) {
        typename Rows::Dist d = rows.open(b, u, N, V, &s_scratch);
        // p_u(x), q_u(x) and the uniform of every sibling are fetched side by side up front, so that the sibling
        // loop below pays for one dependent trip to memory in total instead of one per sibling
        for (int m = tid; m < cnt; m += kVerifyThreads) {
            const int x = s_tok[first + m];
            const bool valid = x >= 0 && x < V;
            s_px[m] = valid ? d.p_of(x) : -1.0;               // -1: no such token, never accepted
            s_qx[m] = valid ? d.q_of(x) : 0.0;
            s_ua[m] = u_accept[(size_t)b * N + first + m];
        }
        __syncthreads();
        double c = 0.0, Y = 1.0;
        for (int m = 0; m < cnt; ++m) {
            const int child = first + m;
            if (tid == 0) {
                double a = 0.0;
                if (s_px[m] >= 0.0) {
                    const double px = s_px[m], qx = s_qx[m];
                    const double num = fmax(px - c * qx, 0.0);
                    a = qx > 0.0 ? fmin(1.0, num / (Y * qx)) : (num > 0.0 ? 1.0 : 0.0);
                }
                s_accept = ((double)s_ua[m] < a) ? 1 : 0;
            }
            __syncthreads();
            const int acc = s_accept;
            __syncthreads();
            if (acc) { st.next_child = child; break; }
            c += Y;
            d.set_c(c);
            Y = dist_mass(d, &s_scratch);
            if (!(Y > 0.0)) { c = 0.0; Y = 1.0; d.set_c(0.0); }     // nothing left: back to the un-residualised row
        }
        if (st.next_child < 0) st.c = c;
    }
    // ---- ticket: the block that finishes a sequence's last node goes on to the select phase
    if (tid == 0) {
        state[(size_t)b * N + u] = st;
        // One acquire-release ticket instead of fence, ticket, fence (three trips to memory in a row on the path of
        // the block that finishes last): the state above is visible before the ticket is, and the block that draws
        // the last ticket sees the states of all the others.
        int old;
        asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(tickets + b) : "memory");
        s_last = (old == n_act - 1) ? 1 : 0;
        if (s_last) *(volatile int*)&tickets[b] = 0;       // nobody else arrives in this launch: ready for the next one
    }
    __syncthreads();
    if (!s_last) return;
    select_and_draw(rows, tokens, state + (size_t)b * N, b, n_levels, n_roots, u_bonus, N, V, accept_len, out_tokens, out_nodes,
                    best_root, next_roots, R, &s_scratch);
}

// Several distinct new tokens from the distribution the winning path stopped with (Section 3.1 samples more than
// one token from the target side to start the next candidate tree): one thread block per sequence, draw i by
// inverse CDF with uniform u_roots[b][i] over the ids not drawn before.  Runs after the two verify kernels on the
// same workspace, from which it takes the stop node's residual coefficient.
template <typename Rows>
__global__ void __launch_bounds__(kVerifyThreads)
sample_roots_kernel(Rows rows, const NodeState* __restrict__ state, const int32_t* __restrict__ accept_len,
                    const int32_t* __restrict__ out_nodes, const int32_t* __restrict__ best_root, int n_levels,
                    const float* __restrict__ u_roots, int N, int V, int R, int32_t* __restrict__ next_roots) {
    using Dist = typename Rows::Dist;
    constexpr int E = Dist::E;
    __shared__ VerifyScratch s_scratch;
    __shared__ CdfScratch s_cdf;
    __shared__ int s_pick[32];
    const int b = blockIdx.x, tid = threadIdx.x;
    const int ln = min(max(accept_len[b], 0), n_levels);
    int u = ln > 0 ? out_nodes[(size_t)b * n_levels + ln - 1] : best_root[b];
    u = min(max(u, 0), N - 1);
    Dist d = rows.open(b, u, N, V, &s_scratch);
    d.set_c(state[(size_t)b * N + u].c);
    for (int i = 0; i < R; ++i) {
        const int* picks = s_pick;
        auto drop = [i, picks](int idx, float (&r)[E]) {
            for (int j = 0; j < i; ++j) {                    // ids already drawn carry no mass any more
                const int e = picks[j] - idx;
#pragma unroll
                for (int k = 0; k < E; ++k)
                    if (e == k) r[k] = 0.f;
            }
        };
        auto load = [&d, &drop](int idx, float (&r)[E]) { d.load(idx, r); drop(idx, r); };
        double total;
        cdf_range_sums_dist(d, drop, V, &s_cdf);
        int tok = cdf_locate<E>(load, (double)u_roots[(size_t)b * R + i], false, V, &s_cdf, &total);
        if (!(total > 0.0)) {                                 // nothing left: the rest of the list is empty
            for (int j = i + tid; j < R; j += kVerifyThreads) next_roots[(size_t)b * R + j] = -1;
            break;
        }
        if (tid == 0) { s_pick[i] = tok; next_roots[(size_t)b * R + i] = tok; }
        __syncthreads();
    }
}

}  // namespace mcsd
