// Tree attention (Section 2.2 of the paper) on the CUDA cores: the path for fp32 tensors and for shapes the
// tensor-core kernel does not take.  Flash-style: key/value tiles are staged in shared memory, every warp
// keeps an online softmax (running maximum, sum and weighted values) for its queries, the keys of one
// (sequence, head) can be split over several thread blocks, and a combine kernel merges the partials.
//
// Key j of sequence b is row j of the prefix cache for j < L_b, else tree node j - L_b, which query n may
// see iff bit (j - L_b) of its ancestor bitset is set.
#include <cuda_bf16.h>

#include "attention.cuh"

namespace mcsd {

constexpr int kSimtThreads = 256;
constexpr int kSimtWarps = kSimtThreads / 32;
constexpr int kSimtQPerWarp = 3;
constexpr int kSimtQBlock = kSimtWarps * kSimtQPerWarp;   // 24 queries per thread block
constexpr int kSimtTile = 32;                             // keys per shared-memory tile

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// 16 bytes of a row as floats: 4 fp32 values or 8 bf16 values (converted in registers)
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int E = 4;
    __device__ __forceinline__ static void load(const float* p, float (&r)[4]) {
        const float4 v = *reinterpret_cast<const float4*>(p);
        r[0] = v.x; r[1] = v.y; r[2] = v.z; r[3] = v.w;
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int E = 8;
    __device__ __forceinline__ static void load(const __nv_bfloat16* p, float (&r)[8]) {
        const uint4 v = *reinterpret_cast<const uint4*>(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {                     // a bf16 is the upper half of the fp32 with the same value
            r[2 * i] = __uint_as_float(w[i] << 16);
            r[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
};

// grid: (splits, query blocks, B * H)
template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads)
tree_attention_simt_kernel(const T* __restrict__ q, const T* __restrict__ k_cache, const T* __restrict__ v_cache,
                           const T* __restrict__ k_tree, const T* __restrict__ v_tree, T* __restrict__ out,
                           const int32_t* __restrict__ seq_lens, const int32_t* __restrict__ n_active,
                           const uint64_t* __restrict__ anc, int words, int H, int G, int N, int L_max, float scale,
                           int splits, float* __restrict__ part_ml, float* __restrict__ part_acc) {
    constexpr int DL = D / 32;                            // output columns per lane
    __shared__ float s_q[kSimtQBlock][D];
    __shared__ float s_k[kSimtTile][D + 1];
    __shared__ float s_v[kSimtTile][D];
    const int bh = blockIdx.z, b = bh / H;
    const int split = blockIdx.x, q0 = blockIdx.y * kSimtQBlock;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int L = min(max(seq_lens[b], 0), L_max);
    const int Nb = n_active ? min(max(n_active[b], 0), N) : N;
    if (q0 >= Nb) return;
    const int total = L + Nb;
    int chunk = (total + splits - 1) / splits;
    chunk = (chunk + kSimtTile - 1) / kSimtTile * kSimtTile;
    const int j_begin = split * chunk, j_end = min(total, j_begin + chunk);

    constexpr int EV = Vec16<T>::E, DV = D / EV;          // elements per 16-byte load, loads per row
    const T* qb = q + (size_t)bh * N * D;
    const size_t bkv = (size_t)b * (H / G) + (bh % H) / G;   // query head h reads key/value head h / G
    const T* kc = k_cache + bkv * L_max * D;
    const T* vc = v_cache + bkv * L_max * D;
    const T* kt = k_tree + bkv * N * D;
    const T* vt = v_tree + bkv * N * D;
    // rows are multiples of 16 bytes long, so 128-bit loads need only 16-byte aligned tensors (uniform per launch)
    const bool vec = ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_cache) | reinterpret_cast<uintptr_t>(v_cache) |
                       reinterpret_cast<uintptr_t>(k_tree) | reinterpret_cast<uintptr_t>(v_tree)) & 15u) == 0;
    if (vec) {
        for (int i = tid; i < kSimtQBlock * DV; i += kSimtThreads) {
            const int r = i / DV, d = (i % DV) * EV;
            float v[EV];
#pragma unroll
            for (int e = 0; e < EV; ++e) v[e] = 0.f;
            if (q0 + r < Nb) Vec16<T>::load(qb + (size_t)(q0 + r) * D + d, v);
#pragma unroll
            for (int e = 0; e < EV; ++e) s_q[r][d + e] = v[e];
        }
    } else {
        for (int i = tid; i < kSimtQBlock * D; i += kSimtThreads) {
            const int r = i / D, d = i % D;
            s_q[r][d] = (q0 + r < Nb) ? to_f32(qb[(size_t)(q0 + r) * D + d]) : 0.f;
        }
    }

    float m[kSimtQPerWarp], l[kSimtQPerWarp], o[kSimtQPerWarp][DL];
#pragma unroll
    for (int i = 0; i < kSimtQPerWarp; ++i) {
        m[i] = -INFINITY; l[i] = 0.f;
#pragma unroll
        for (int c = 0; c < DL; ++c) o[i][c] = 0.f;
    }

    for (int j0 = j_begin; j0 < j_end; j0 += kSimtTile) {
        __syncthreads();
        if (vec) {
            // one 128-bit load of K and one of V per thread and step, converted in registers
            for (int i = tid; i < kSimtTile * DV; i += kSimtThreads) {
                const int r = i / DV, d = (i % DV) * EV, j = j0 + r;
                float kv[EV], vv[EV];
#pragma unroll
                for (int e = 0; e < EV; ++e) { kv[e] = 0.f; vv[e] = 0.f; }
                if (j < j_end) {
                    const T* kr = j < L ? kc + (size_t)j * D : kt + (size_t)(j - L) * D;
                    const T* vr = j < L ? vc + (size_t)j * D : vt + (size_t)(j - L) * D;
                    Vec16<T>::load(kr + d, kv);
                    Vec16<T>::load(vr + d, vv);
                }
#pragma unroll
                for (int e = 0; e < EV; ++e) { s_k[r][d + e] = kv[e]; s_v[r][d + e] = vv[e]; }
            }
        } else {
            for (int i = tid; i < kSimtTile * D; i += kSimtThreads) {
                const int r = i / D, d = i % D, j = j0 + r;
                float kv = 0.f, vv = 0.f;
                if (j < j_end) {
                    if (j < L) { kv = to_f32(kc[(size_t)j * D + d]); vv = to_f32(vc[(size_t)j * D + d]); }
                    else { kv = to_f32(kt[(size_t)(j - L) * D + d]); vv = to_f32(vt[(size_t)(j - L) * D + d]); }
                }
                s_k[r][d] = kv;
                s_v[r][d] = vv;
            }
        }
        __syncthreads();
        const int j = j0 + lane;                          // this lane's key
#pragma unroll
        for (int i = 0; i < kSimtQPerWarp; ++i) {
            const int n = q0 + warp * kSimtQPerWarp + i;
            if (n >= Nb) continue;                        // uniform per warp
            bool ok = j < j_end;
            if (ok && j >= L) {
                const int t = j - L;
                ok = (anc[(size_t)n * words + (t >> 6)] >> (t & 63)) & 1ull;
            }
            float s = 0.f;
#pragma unroll 8
            for (int d = 0; d < D; ++d) s = fmaf(s_q[warp * kSimtQPerWarp + i][d], s_k[lane][d], s);
            s = ok ? s * scale : -INFINITY;
            float mx = s;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
            const float m_new = fmaxf(m[i], mx);
            if (m_new == -INFINITY) continue;             // nothing visible yet (uniform per warp)
            const float alpha = expf(m[i] - m_new);       // exp(-inf) = 0 on the first visible tile
            const float pj = ok ? expf(s - m_new) : 0.f;
            float ps = pj;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, off);
            l[i] = l[i] * alpha + ps;
            m[i] = m_new;
#pragma unroll
            for (int c = 0; c < DL; ++c) o[i][c] *= alpha;
            for (int kk = 0; kk < kSimtTile; ++kk) {
                const float pk = __shfl_sync(0xffffffffu, pj, kk);
#pragma unroll
                for (int c = 0; c < DL; ++c) o[i][c] = fmaf(pk, s_v[kk][lane + 32 * c], o[i][c]);
            }
        }
    }

#pragma unroll
    for (int i = 0; i < kSimtQPerWarp; ++i) {
        const int n = q0 + warp * kSimtQPerWarp + i;
        if (n >= Nb) continue;
        if (splits == 1) {
            const float inv = l[i] > 0.f ? 1.f / l[i] : 0.f;
            T* dst = out + ((size_t)bh * N + n) * D;
#pragma unroll
            for (int c = 0; c < DL; ++c) dst[lane + 32 * c] = from_f32<T>(o[i][c] * inv);
        } else {
            const size_t slot = ((size_t)bh * splits + split) * N + n;
            if (lane == 0) { part_ml[2 * slot] = m[i]; part_ml[2 * slot + 1] = l[i]; }
#pragma unroll
            for (int c = 0; c < DL; ++c) part_acc[slot * D + lane + 32 * c] = o[i][c];
        }
    }
}

// grid: (N, B * H); one warp merges the partials of one query
template <typename T, int D>
__global__ void __launch_bounds__(32)
tree_attention_simt_combine_kernel(T* __restrict__ out, const int32_t* __restrict__ n_active, int H, int N, int splits,
                                   const float* __restrict__ part_ml, const float* __restrict__ part_acc) {
    constexpr int DL = D / 32;
    const int bh = blockIdx.y, b = bh / H, n = blockIdx.x, lane = threadIdx.x;
    const int Nb = n_active ? min(max(n_active[b], 0), N) : N;
    if (n >= Nb) return;
    float M = -INFINITY;
    for (int s = 0; s < splits; ++s) M = fmaxf(M, part_ml[2 * (((size_t)bh * splits + s) * N + n)]);
    float lsum = 0.f, acc[DL];
#pragma unroll
    for (int c = 0; c < DL; ++c) acc[c] = 0.f;
    for (int s = 0; s < splits; ++s) {
        const size_t slot = ((size_t)bh * splits + s) * N + n;
        const float ms = part_ml[2 * slot];
        if (ms == -INFINITY) continue;
        const float w = expf(ms - M);
        lsum += w * part_ml[2 * slot + 1];
#pragma unroll
        for (int c = 0; c < DL; ++c) acc[c] = fmaf(w, part_acc[slot * D + lane + 32 * c], acc[c]);
    }
    const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
    T* dst = out + ((size_t)bh * N + n) * D;
#pragma unroll
    for (int c = 0; c < DL; ++c) dst[lane + 32 * c] = from_f32<T>(acc[c] * inv);
}

static int simt_splits(int B, int H, int N, int L_max) {
    const int qblocks = (N + kSimtQBlock - 1) / kSimtQBlock;
    const long long ctas = (long long)B * H * qblocks;
    const int want = (int)((148LL * 8 + ctas - 1) / ctas);            // about eight blocks per SM
    const int max_splits = (L_max + N + 4 * kSimtTile - 1) / (4 * kSimtTile);
    int s = want < 1 ? 1 : want;
    if (s > max_splits) s = max_splits;
    if (s > 64) s = 64;
    return s < 1 ? 1 : s;
}

size_t simt_workspace_bytes(int B, int H, int N, int D, int L_max) {
    const int s = simt_splits(B, H, N, L_max);
    if (s == 1) return 0;
    const size_t slots = (size_t)B * H * s * N;
    return align_up(slots * 2 * sizeof(float), 256) + align_up(slots * D * sizeof(float), 256);
}

template <typename T, int D>
static int launch_simt(const AttentionArgs& a, void* scratch, cudaStream_t stream) {
    const int splits = simt_splits(a.B, a.H, a.N, a.L_max);
    const size_t slots = (size_t)a.B * a.H * splits * a.N;
    float* part_ml = static_cast<float*>(scratch);
    float* part_acc = reinterpret_cast<float*>(static_cast<char*>(scratch) + align_up(slots * 2 * sizeof(float), 256));
    const int qblocks = (a.N + kSimtQBlock - 1) / kSimtQBlock;
    dim3 grid(splits, qblocks, a.B * a.H);
    tree_attention_simt_kernel<T, D><<<grid, kSimtThreads, 0, stream>>>(
        static_cast<const T*>(a.q), static_cast<const T*>(a.k_cache), static_cast<const T*>(a.v_cache),
        static_cast<const T*>(a.k_tree), static_cast<const T*>(a.v_tree), static_cast<T*>(a.out), a.seq_lens,
        a.n_active, a.anc, a.words, a.H, a.G, a.N, a.L_max, a.scale, splits, part_ml, part_acc);
    MCSD_CUDA_CHECK(cudaGetLastError());
    count_launches(1);
    if (splits > 1) {
        tree_attention_simt_combine_kernel<T, D><<<dim3(a.N, a.B * a.H), 32, 0, stream>>>(
            static_cast<T*>(a.out), a.n_active, a.H, a.N, splits, part_ml, part_acc);
        MCSD_CUDA_CHECK(cudaGetLastError());
        count_launches(1);
    }
    return MCSD_OK;
}

int tree_attention_simt(const AttentionArgs& a, void* scratch, cudaStream_t stream) {
    if (a.dtype == MCSD_F32) {
        return a.D == 64 ? launch_simt<float, 64>(a, scratch, stream) : launch_simt<float, 128>(a, scratch, stream);
    }
    return a.D == 64 ? launch_simt<__nv_bfloat16, 64>(a, scratch, stream)
                     : launch_simt<__nv_bfloat16, 128>(a, scratch, stream);
}

}  // namespace mcsd
