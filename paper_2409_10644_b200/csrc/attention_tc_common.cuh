// Pieces of the tcgen05 tree-attention kernel (Section 2.2 of the paper) that are not its main loop: launch parameters, inline-PTX
// wrappers (mbarrier, TMA, tcgen05), and the bookkeeping that cuts the flattened (sequence, head, query block,
// key tile) space into per-block ranges of equal cost.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>

#include "attention.cuh"

namespace mcsd {

constexpr int kTile = 128;                    // keys per tile
constexpr int kSlotBytes = kTile * 128 * 2;   // one K or V tile: 128 rows x 128 bf16
constexpr int kSlabBytes = kTile * 128;       // 64 of the 128 columns: rows of 128 bytes (the TMA swizzle span)
constexpr int kMaxSlots = 6;
constexpr int kMaxBatchTc = 256;
constexpr int kTmemCols = 512;
constexpr float kLazyTau = 8.0f;              // raise the reference maximum only beyond 2^8
constexpr int kMaxCtas = 160;                 // partial slots are provisioned for this many thread blocks
constexpr int kMaxParts = kMaxCtas;           // a work item is cut into at most one piece per thread block
constexpr int kMaxQ = 160;                    // queries per work item in the widest instantiation (stride of the partials)
constexpr long long kSpinCycles = 4000000000LL;   // about two seconds
constexpr int kSmemLimit = 232448;            // dynamic shared memory a block may opt in to

// Tiles and cost of the sequences before b, per head.
struct TileIndex {
    int cum_tiles[kMaxBatchTc + 1];
    int cum_w[kMaxBatchTc + 1];
    unsigned short kv_tiles[kMaxBatchTc];   // key tiles of one work item of sequence b
    int whole_items;                        // launch small enough to give every block whole work items (see plan_ranges)
    int scan[kMaxBatchTc / 32][4];          // per-warp totals of plan_ranges' scan
    int len[kMaxBatchTc];                   // clamped prefix length of sequence b
    unsigned short nodes[kMaxBatchTc];      // clamped active tree nodes of sequence b
};
constexpr int kWholeItemTiles = 8;          // ... which pays while a work item has at most this many key tiles

struct TcParams {
    __nv_bfloat16* out;
    const int32_t* seq_lens;
    const int32_t* n_active;
    const uint64_t* anc;
    int words;
    int B, H, N, L_max;      // H: work units per sequence = query heads / G; N tree nodes (= tree keys)
    int G, g_shift;          // query heads stacked into one work unit (1, 2, 4 or 8 = 1 << g_shift): its G * N queries
                             // are taken node-major, query j = head j % G of the unit, node j / G
    int Hkv, group;          // key/value heads, and query heads per key/value head (a multiple of G): unit u of a
                             // sequence reads key/value head u * G / group
    float scale_log2;
    float* part_ml;      // [2 * kMaxCtas][2][kMaxQ]
    float* part_o;       // [2 * kMaxCtas][kMaxQ][128]
    int* counters;       // [B * H][query block][softmax group] arrivals per split work item; zero between launches
    WorkspaceHeader* header;
    int n_slots;
    int npadq;           // rows of the Q box = 16 * (template chunk count)
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(void* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(void* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(void* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(void* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false if the wait ran out or another role already gave up (abort_flag, in shared memory);
// `where` names the wait in the workspace header.
static __device__ __noinline__ bool mbar_wait_slow(void* bar, uint32_t parity, int* abort_flag, WorkspaceHeader* header, int where,
                                                   long long limit = kSpinCycles) {
    const long long t0 = clock64();
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u) {
            if (*(volatile int*)abort_flag) return false;
            if (clock64() - t0 > limit) {
                *(volatile int*)abort_flag = 1;
                header->detail = where;
                header->status = MCSD_ERR_TIMEOUT;
                __threadfence();
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(void* bar, uint32_t parity, int* abort_flag, WorkspaceHeader* header, int where) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, header, where);
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, void* bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z) : "memory");
}

// The same load with an L2 eviction-priority hint (from createpolicy): the key/value stream is read once and should
// not push the split-KV partials, which are read back at the end of the kernel, out of L2.
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap* map, void* bar, int x, int y, int z, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
        ::"r"(dst), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, void* bar, int x, int y, int z, int w) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// tcgen05.mma and tcgen05.commit for a warp that executes them convergently: one elected lane issues.  (The lane that
// issued the MMAs must also issue the commit that tracks them; elect.sync picks the same lane every time.)
__device__ __forceinline__ void tc_mma_elect(uint32_t d_tmem, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p, e;\n\t"
        "elect.sync _|e, 0xffffffff;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit_elect(void* bar) {
    asm volatile(
        "{\n\t.reg .pred e;\n\t"
        "elect.sync _|e, 0xffffffff;\n\t"
        "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(smem_u32(bar)) : "memory");
}
// eight consecutive fp32 columns of this thread's TMEM lane; the caller waits with tc_wait_ld()
__device__ __forceinline__ void tc_ld8(uint32_t taddr, float* v) {
    uint32_t r[8];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
// four consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tc_ld4(uint32_t taddr, float* v) {
    uint32_t r[4];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ float tc_ld1(uint32_t taddr) {
    float v;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=f"(v) : "r"(taddr) : "memory");
    return v;
}
__device__ __forceinline__ void tc_st1(uint32_t taddr, float v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x1.b32 [%0], {%1};" ::"r"(taddr), "f"(v) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_st8(uint32_t taddr, const float* v) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
        ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
          "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
          "r"(__float_as_uint(v[7])) : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float warp_max_f32(float v) {
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}
// named barrier `id` over the 128 threads of one softmax warpgroup, returning the OR of `pred`
__device__ __forceinline__ bool group_sync_any(int id, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %2, 0;\n\t"
        "bar.red.or.pred q, %1, 128, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"(id), "r"((uint32_t)pred) : "memory");
    return r != 0;
}

// Shared-memory matrix descriptor of tcgen05.mma: start address, leading/stride byte offsets (all >> 4),
// descriptor version 1, swizzle mode in the top bits (0 = none, 2 = 128-byte).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | ((uint64_t)layout << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, M = 128, N = n, operand major-ness.
__device__ __forceinline__ uint32_t instr_desc(int n, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// ------------------------------------------------------------------ tile bookkeeping
// Queries are processed in blocks of at most QB (the tensor-memory budget: 128, or 160 in the widest kernel); a
// tree with more stacked queries makes each (sequence, head) two work items that read the same keys.  Tiles per
// work item: prefix tiles, then tree tiles.  Everything below is a pure function of the launch so that all thread
// blocks cut the tile space alike.
__host__ __device__ __forceinline__ int kv_tiles_of(int L, int Nb) {
    return Nb > 0 ? (L + kTile - 1) / kTile + (Nb + kTile - 1) / kTile : 0;
}
template <int QB>
__host__ __device__ __forceinline__ int tiles_of(int L, int Nb, int G) {
    return kv_tiles_of(L, Nb) * ((Nb * G + QB - 1) / QB);
}

struct Segment {
    int b, h, lt, Tb, L, Nb, nP;
    int qb, q0, Nq, Tkv;      // query block, its first query, its query count, tiles per query block
};

template <int QB>
__host__ __device__ __forceinline__ void locate(const TileIndex* ix, const TcParams& p, long long t, Segment& s) {
    int lo = 0, hi = p.B;                      // find b with H*cum[b] <= t < H*cum[b+1]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((long long)p.H * ix->cum_tiles[mid] <= t) lo = mid; else hi = mid;
    }
    s.b = lo;
    s.L = ix->len[lo];
    s.Nb = ix->nodes[lo];
    s.Tb = ix->cum_tiles[lo + 1] - ix->cum_tiles[lo];
    s.nP = (s.L + kTile - 1) / kTile;
    const long long r = t - (long long)p.H * ix->cum_tiles[lo];
    int rem;
    if ((unsigned long long)r >> 32) {                 // 64-bit division only where it is needed
        s.h = (int)(r / s.Tb);
        rem = (int)(r % s.Tb);
    } else {
        const uint32_t r32 = (uint32_t)r, h32 = r32 / (uint32_t)s.Tb;
        s.h = (int)h32;
        rem = (int)(r32 - h32 * (uint32_t)s.Tb);
    }
    s.Tkv = kv_tiles_of(s.L, s.Nb);
    if (s.Tb == s.Tkv) {                               // one query block
        s.qb = 0;
        s.lt = rem;
    } else {
        s.qb = rem / s.Tkv;
        s.lt = rem - s.qb * s.Tkv;
    }
    s.q0 = s.qb * QB;
    s.Nq = min(QB, s.Nb * p.G - s.q0);
}

// Cost of one tile and fixed cost of a work item in units of 32 ns: a least-squares fit of the time thread blocks
// were busy (device clock stamps, the wide workloads with several seeds each) against the tiles, work items and
// query counts they had been given.  Thread blocks get equal cost, not equal tile counts, so that sequences with
// deep trees do not make their blocks finish late.  At most 64 per tile and 256 per work item (the launch bound on
// the 32-bit prefix sums counts on it).
template <int QB>
__host__ __device__ __forceinline__ int tile_weight(int Nq) { return (QB > 128 ? 34 : 29) + (Nq * 83 + (Nq * Nq * 35) / 64) / 1024; }
// Fixed cost of a work item (the wait for the last product, normalisation and output of Nq columns, locating the
// next item).  The fit puts it at the item's end, so the item's last tile carries it: a block that takes only the
// first tiles of an item does not pay it.
template <int QB>
__host__ __device__ __forceinline__ int item_weight(int Nq) { return QB > 128 ? 119 + (Nq * 130) / 256 : 109 + (Nq * 47) / 256; }
template <int QB>
__host__ __device__ __forceinline__ int head_weight(int L, int Nk, int G) {  // cost of one (sequence, head): all query blocks
    const int tkv = kv_tiles_of(L, Nk);
    const int Nb = Nk * G;                                        // stacked queries
    int w = 0;
    for (int q0 = 0; q0 < Nb; q0 += QB) w += tkv * tile_weight<QB>(min(QB, Nb - q0)) + item_weight<QB>(min(QB, Nb - q0));
    return w;
}
// cumulative cost of the tiles before the one a Segment points at
template <int QB>
__host__ __device__ __forceinline__ long long weight_before(const TileIndex* ix, const TcParams& p, const Segment& s) {
    long long w = (long long)p.H * ix->cum_w[s.b] + (long long)s.h * (ix->cum_w[s.b + 1] - ix->cum_w[s.b]);
    if (s.qb) w += (long long)s.Tkv * tile_weight<QB>(QB) + item_weight<QB>(QB);
    return w + (long long)s.lt * tile_weight<QB>(s.Nq);
}
// Tile t belongs to block floor(weight_before(t) * G / total_w).  First tile of block c: the first tile whose
// cumulative cost reaches ceil(c * total_w / G).
template <int QB>
__host__ __device__ __forceinline__ long long first_tile_of_block(const TileIndex* ix, const TcParams& p, int c, int G, long long total_w,
                                                         long long total_tiles) {
    const long long wt = ((long long)c * total_w + G - 1) / G;
    if (wt >= total_w) return total_tiles;
    int lo = 0, hi = p.B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((long long)p.H * ix->cum_w[mid] <= wt) lo = mid; else hi = mid;
    }
    const int L = min(max(p.seq_lens[lo], 0), p.L_max);
    const int Nk = p.n_active ? min(max(p.n_active[lo], 0), p.N) : p.N;
    const int tkv = kv_tiles_of(L, Nk);
    const int Nb = Nk * p.G;                                      // stacked queries
    const int wh = ix->cum_w[lo + 1] - ix->cum_w[lo], tb = ix->cum_tiles[lo + 1] - ix->cum_tiles[lo];
    const long long rem = wt - (long long)p.H * ix->cum_w[lo];
    const int h = (int)(rem / wh);
    int r2 = (int)(rem % wh);
    long long t = (long long)p.H * ix->cum_tiles[lo] + (long long)h * tb;
    // inside a work item tile k starts at cost k * w; the last tile also carries the fixed cost, so a cost beyond the
    // start of the last tile is reached only by the first tile of what follows
    int w = tile_weight<QB>(min(QB, Nb));
    const int item0 = tkv * w + item_weight<QB>(min(QB, Nb));
    if (Nb > QB && r2 >= item0) {                      // inside the second query block
        r2 -= item0;
        t += tkv;
        w = tile_weight<QB>(Nb - QB);
    }
    return t + min(tkv, (r2 + w - 1) / w);
}
template <int QB>
__host__ __device__ __forceinline__ int block_of_tile(const TileIndex* ix, const TcParams& p, long long t, int G, long long total_w) {
    Segment s;
    locate<QB>(ix, p, t, s);
    return (int)min((long long)G - 1, weight_before<QB>(ix, p, s) * G / total_w);
}

// Per-sequence entries of the tile index (the prefix sums over sequences are the caller's).
template <int QB>
__host__ __device__ __forceinline__ void plan_sequence(TileIndex* ix, const TcParams& p, int b, int& tiles, int& cost, int& items,
                                                       int& kv) {
    const int L = min(max(p.seq_lens[b], 0), p.L_max);
    const int Nb = p.n_active ? min(max(p.n_active[b], 0), p.N) : p.N;
    kv = min(kv_tiles_of(L, Nb), 65535);
    tiles = tiles_of<QB>(L, Nb, p.G);
    cost = head_weight<QB>(L, Nb, p.G);
    items = Nb > 0 ? (Nb * p.G + QB - 1) / QB : 0;          // query blocks of the sequence
    ix->kv_tiles[b] = (unsigned short)kv;
    ix->len[b] = L;
    ix->nodes[b] = (unsigned short)Nb;
}
// How many blocks get work, and in which mode, once the prefix sums are in place.
template <int QB>
__host__ __device__ __forceinline__ int plan_blocks(TileIndex* ix, const TcParams& p, int grid, int items, int longest) {
    // Few short work items (one sequence with a short prefix, say): a block's fixed costs outweigh its tiles, and
    // cutting items into pieces would add a partial and a merge to each.  Every block then takes whole items.
    const long long n_items = (long long)p.H * items;
    ix->whole_items = (n_items > 0 && n_items <= (long long)grid && longest <= kWholeItemTiles) ? 1 : 0;
    // Otherwise no block's share of the cost may be smaller than the heaviest tile, so that consecutive tiles never
    // skip a block: every working block then owns at least one tile and the blocks sharing a work item are
    // consecutive.
    const long long tot_w = (long long)p.H * ix->cum_w[p.B];
    return ix->whole_items ? (int)n_items
                           : (int)max(1LL, min((long long)grid, tot_w / (tile_weight<QB>(QB) + item_weight<QB>(QB))));
}
// First tile of block c of nb (c == nb: one past the last tile).
template <int QB>
__host__ __device__ __forceinline__ long long range_start(const TileIndex* ix, const TcParams& p, int c, int nb) {
    const long long tot = (long long)p.H * ix->cum_tiles[p.B], tot_w = (long long)p.H * ix->cum_w[p.B];
    if (tot <= 0 || c >= nb) return tot > 0 ? tot : 0;
    if (!ix->whole_items) return first_tile_of_block<QB>(ix, p, c, nb, tot_w, tot);
    // first tile of work item number c = (sequence, head, query block) in tile order
    for (int b = 0; b < p.B; ++b) {
        const int kv = ix->kv_tiles[b], tb = ix->cum_tiles[b + 1] - ix->cum_tiles[b];
        const int per_seq = kv > 0 ? p.H * (tb / kv) : 0;
        if (c < per_seq) return (long long)p.H * ix->cum_tiles[b] + (long long)c * kv;
        c -= per_seq;
    }
    return tot;
}

// Per-block set-up: tiles and cost per sequence, their prefix sums, the number of blocks that get work and the two
// ends of this block's range.  Ends with a __syncthreads(); all threads must call it.
template <int QB>
__device__ __forceinline__ void plan_ranges(TileIndex* ix, const TcParams& p, int* n_blocks, long long* range) {
    const int tid = threadIdx.x, lane = tid & 31, wrp = tid >> 5;
    // thread b < B owns sequence b (B <= 256 <= blockDim.x): its tiles, cost and work items, then an inclusive scan
    // over the sequences, by warp shuffles and one exchange of the eight warp totals
    int v_t = 0, v_w = 0, v_i = 0, v_kv = 0;
    if (tid < kMaxBatchTc) {
        if (tid < p.B) plan_sequence<QB>(ix, p, tid, v_t, v_w, v_i, v_kv);
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int a = __shfl_up_sync(0xffffffffu, v_t, o), c = __shfl_up_sync(0xffffffffu, v_w, o),
                      d = __shfl_up_sync(0xffffffffu, v_i, o);
            if (lane >= o) { v_t += a; v_w += c; v_i += d; }
        }
        v_kv = __reduce_max_sync(0xffffffffu, v_kv);
        if (lane == 31) { ix->scan[wrp][0] = v_t; ix->scan[wrp][1] = v_w; ix->scan[wrp][2] = v_i; ix->scan[wrp][3] = v_kv; }
    }
    __syncthreads();
    if (tid < kMaxBatchTc) {
        int items = 0, longest = 0;
        for (int x = 0; x < kMaxBatchTc / 32; ++x) {
            if (x < wrp) { v_t += ix->scan[x][0]; v_w += ix->scan[x][1]; }
            items += ix->scan[x][2];
            longest = max(longest, ix->scan[x][3]);
        }
        if (tid < p.B) { ix->cum_tiles[tid + 1] = v_t; ix->cum_w[tid + 1] = v_w; }
        if (tid == 0) { ix->cum_tiles[0] = 0; ix->cum_w[0] = 0; }
        // the thread that wrote the totals (plan_blocks reads only cum_w[B])
        if (tid == max(p.B, 1) - 1) *n_blocks = plan_blocks<QB>(ix, p, (int)gridDim.x, items, longest);
    }
    __syncthreads();
    if (tid == 0 || tid == 32) {               // the two ends of this block's range, side by side
        const int which = tid >> 5;
        range[which] = (int)blockIdx.x < *n_blocks ? range_start<QB>(ix, p, (int)blockIdx.x + which, *n_blocks) : 0;
    }
    __syncthreads();
}

struct TcLaunch {
    CUtensorMap maps[9];     // Q, key cache, value cache, tree keys, tree values; the last four again in boxes of 64 rows
    TcParams p;
    int grid;
};

}  // namespace mcsd
