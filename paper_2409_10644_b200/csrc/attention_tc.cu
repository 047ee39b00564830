// Tree attention (Section 2.2 of the paper) on the fifth-generation tensor cores of sm_100a: bf16, head_dim 128,
// 1 to 160 query columns per work item in one pass over the keys (narrow static trees up to the paper's
// many-candidate regime: fork width 16 and more, the target-initialised forests of Section 3.1).
//
// One persistent thread block per SM walks a contiguous range of 128-key tiles of the flattened
// (sequence, head, query block, key tile) space, so the K/V stream of every (sequence, head) is read from HBM once
// and all SMs carry the same cost whatever the batch and the prefix lengths are.  Where a range boundary cuts a
// work item, the blocks that continue it write unnormalised partials (reference, sum, weighted values) as the
// first thing they do and take a ticket; the block that started the item, whose piece is its last segment and is
// still in tensor memory, folds them in at its end: split-KV with a fused combine.
//
// The problem is set up transposed so that the small dimension (tree tokens) is the MMA N and the 128 keys of a
// tile fill the MMA M:
//     S^T[key][query] = K_tile * Q^T,   O^T[d][query] += V_tile^T * P^T,   l[query] += P * 1
// (A = K tile and B = Q K-major from TMA; A = V tile read MN-major, B = P^T written MN-major by the softmax
// threads).  Tensor memory: S^T twice (columns 0, 160), O^T (320), row sums (480 for queries 0..127, 496 for queries
// 128..159) = all 512 columns.
//
// How the work is organised:
//   * three softmax warpgroups (12 warps, 128 registers per thread) split the query columns of every tile; thread r
//     of a group owns key row r of the tile = TMEM lane r.  Measured against two groups (168 registers) and four
//     (96 registers, spills) on the wide workloads, three is fastest;
//   * the probabilities of a tile are produced in one optimistic sweep (scores shifted by the running reference,
//     checked against the lazy threshold 2^8, exponentiated, packed to bf16 in registers, tensor memory read two
//     column groups per round trip); only when the vote of a group fires are exact column maxima reduced
//     (redux.sync inside a warp, shared memory across warps), O^T and l rescaled and the sweep redone;
//   * row sums come from the tensor cores (P^T read as an MN-major A operand against a matrix of ones) and are
//     accumulated in tensor memory across the tiles of a segment like O^T; they are touched by a thread only when
//     the reference moves and in the epilogue;
//   * the reference of a segment starts from the scores of one key of its first full tile (key 0, 32, 64 or 96,
//     depending on the column group) instead of an exact column maximum: any reference that no score exceeds by
//     more than 2^8 gives the same result, and a key that does exceed it raises the vote like anywhere else.
//     (Segments that start on a ragged or tree tile take the exact path.)
//   * the MMA warp runs its loop convergently and one elected lane issues; descriptors are built once and advanced
//     by constants, and there are two commits per tile (S^T done = scores ready and key slot free; products done =
//     value slot and P^T free), because a tcgen05.mma of these shapes takes 40-60 cycles and the instructions
//     between two of them would otherwise pace the tensor pipe;
//   * the producer issues loads in the order in which slots come free (K0 K1 V0 K2 V1 ...), about two tiles ahead;
//     a tile with at most 64 rows in use is fetched as one 64-row box;
//   * prefix tiles need no mask (a dead key row of a ragged tile is one thread's own row); tree tiles mask the packed
//     probabilities with masks grown from the transposed ancestor bitsets by a multiply and a byte permute.
//
// Warp roles (512 threads): warps 0-11 softmax / mask / epilogue, warp 12 TMA producer, warp 13 MMA issuer and owner
// of the tensor-memory allocation, warp 14 polls the tickets of a split last work item and fetches its first
// partial, warp 15 publishes the partial this block writes; at the end of the block all sixteen warps together
// merge a split item.  Every wait is bounded; one that runs out raises a flag in the workspace header, all roles
// drain and the block exits cleanly.
#include <algorithm>
#include <mutex>
#include <type_traits>

#include "attention_tc_common.cuh"

namespace mcsd {

constexpr int kGroups = 3;                          // softmax warpgroups
constexpr int kProducerWarp = 4 * kGroups, kMmaWarp = kProducerWarp + 1;   // service warpgroup: warps 12..15
constexpr int kTcThreads = 32 * (kProducerWarp + 4);
constexpr int kColS1 = 160, kColO = 320, kColL = 480, kColL2 = 496;
constexpr int kSlots = 4;                      // ring slots that fit next to Q and P^T of 112..160 queries

struct TcSmall {
    unsigned long long slot_full[kSlots];   // [0], [1]: key tile of even / odd tiles, [2], [3]: value tile
    unsigned long long s_full[2];            // S^T of even / odd tiles finished: scores ready, key slot and (last tile) Q free
    unsigned long long pv_done[2];           // products of even / odd tiles finished: value slot and P^T free, O^T and l current
    unsigned long long p_full, q_full, drain;
    unsigned long long merge_bar;            // a staged copy of another block's partial has landed
    unsigned long long s_last;               // the block's last S^T has finished: key slots and Q buffer are free
    int merge_np1;                           // pieces of later blocks to fold into this block's last segment (0: none)
    int merge_prefetched;                    // the first of those pieces is already on its way into shared memory
    Segment merge_item;                      // that segment's work item
    uint32_t tmem_base;
    int abort_flag;
    long long range[2];
    int n_blocks;
    alignas(16) float m_ref[kGroups][64];  // running reference of a group's own query columns (at most 56)
    alignas(16) float alpha[kGroups][64];  // rescale factors of a slow-path tile; in the epilogue 1/l (or l)
    alignas(16) float wred[kGroups][4][64];
    alignas(16) unsigned long long dmask[MCSD_MAX_NODES][3];   // transposed ancestor bitsets
    TileIndex ix;
    alignas(128) __nv_bfloat16 ones[256];   // 16 x 16 matrix of ones: B operand of the row-sum product
};
static_assert(kMaxCtas == kTcMaxBlocks, "the plan's public limit is the kernel's");
static_assert(sizeof(TcSmall) <= kSmemLimit - 1024 - kSlots * 32768 - 160 * 512, "TcSmall grew: four ring slots no longer fit");

// rows of a key/value tile that are fetched when `valid` of them are in use: all 128, or a box of 64
__device__ __forceinline__ int loaded_rows(int valid) { return valid > 64 ? kTile : 64; }
// byte permute; a selector nibble with its top bit set replicates the sign bit of the selected byte
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ uint32_t max_u16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.u16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// 64 bits of a 192-bit row starting at bit `start` (bits past the row read as zero)
__device__ __forceinline__ unsigned long long bits_from(const unsigned long long* w, int start) {
    const int wi = start >> 6, sh = start & 63;
    unsigned long long lo = w[wi] >> sh;
    if (sh != 0 && wi < 2) lo |= w[wi + 1] << (64 - sh);
    return lo;
}

template <int NCH>
__global__ void __launch_bounds__(kTcThreads, 1)
tree_attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kc,
                              const __grid_constant__ CUtensorMap tm_vc, const __grid_constant__ CUtensorMap tm_kt,
                              const __grid_constant__ CUtensorMap tm_vt, const __grid_constant__ CUtensorMap tm_kc64,
                              const __grid_constant__ CUtensorMap tm_vc64, const __grid_constant__ CUtensorMap tm_kt64,
                              const __grid_constant__ CUtensorMap tm_vt64, const TcParams p) {
    static_assert(NCH == 3 || NCH == 4 || NCH == 7 || NCH == 8 || NCH == 10, "padded query columns: 48, 64, 112, 128 or 160");
    constexpr int QB = NCH == 10 ? kMaxQ : 128;    // queries per work item
    constexpr int CPT = (2 * NCH + kGroups - 1) / kGroups; // 8-column groups per thread, at most
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char* ring = smem;                  // four 32 KB slots: keys of even / odd tiles, values of even / odd tiles
    unsigned char* p_buf = ring + (size_t)kSlots * kSlotBytes;
    unsigned char* q_buf = p_buf + (size_t)p.npadq * 256;
    TcSmall* sm = reinterpret_cast<TcSmall*>(q_buf + (size_t)p.npadq * 256);
    const TileIndex* ix = &sm->ix;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;

    // ---- set-up
    // Programmatic dependent launch: a launch that follows this one in the stream may start its blocks as soon as
    // this grid's blocks leave their multiprocessors, and this grid may have been started that way itself.  What
    // comes before the wait below touches no global memory, so it overlaps the tail of the preceding kernel.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // The value slots start out finite: rows of a slot that a partial fetch leaves alone are multiplied by zero
    // probabilities, and 0 * NaN would be NaN.
    for (int i = tid; i < 2 * kSlotBytes / 16; i += kTcThreads)
        reinterpret_cast<uint4*>(ring + 2 * (size_t)kSlotBytes)[i] = make_uint4(0, 0, 0, 0);
    fence_async_smem();                          // ordered before the bulk copies that will write the slots
    if (tid < 256) {
        sm->ones[tid] = __float2bfloat16_rn(1.0f);
        fence_async_smem();                      // read by the tensor cores through the async proxy
    }
    if (tid == 0) {
        for (int i = 0; i < kSlots; ++i) mbar_init(&sm->slot_full[i], 1);
        mbar_init(&sm->s_full[0], 1);
        mbar_init(&sm->s_full[1], 1);
        mbar_init(&sm->pv_done[0], 1);
        mbar_init(&sm->pv_done[1], 1);
        mbar_init(&sm->p_full, 4 * kGroups);      // one arrival per softmax warp
        mbar_init(&sm->q_full, 1);
        mbar_init(&sm->drain, 1);
        mbar_init(&sm->merge_bar, 1);
        mbar_init(&sm->s_last, 1);
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // everything the preceding kernel in the stream wrote is visible from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");
    plan_ranges<QB>(&sm->ix, p, &sm->n_blocks, sm->range);
    const long long total_w = (long long)p.H * ix->cum_w[p.B];
    const int G = sm->n_blocks;
    const long long t_begin = sm->range[0], t_end = sm->range[1];
    if (t_begin >= t_end) return;              // uniform for the whole block: nothing allocated yet

    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *(volatile uint32_t*)&sm->tmem_base;
    WorkspaceHeader* hdr = p.header;
    int* const abort_flag = &sm->abort_flag;

    if (warp == kProducerWarp) {
        // =========================================================== TMA producer
        // Tiles of this block are numbered n = 0, 1, ... across its segments.  Key tile n goes to slot n & 1 as soon
        // as S^T of tile n - 2 has finished, value tile n to slot 2 + (n & 1) as soon as the products of tile n - 2
        // have; loads are issued in the order in which their slots come free (K0 K1 V0 K2 V1 K3 ...), which keeps
        // about two tiles in flight.  Each of these waits targets the latest completion its barrier can have
        // reached (the next one needs the very tile being loaded), so a parity test cannot alias.
        if (lane == 0) {
            const uint32_t total_n = (uint32_t)(t_end - t_begin);
            struct Cursor { long long t; Segment s; int i, cnt; };
            auto open = [&](Cursor& c) {
                locate<QB>(ix, p, c.t, c.s);
                c.cnt = (int)min((long long)(c.s.Tkv - c.s.lt), t_end - c.t);
                c.i = 0;
            };
            Cursor ck, cv;
            ck.t = cv.t = t_begin;
            open(ck);
            cv = ck;
            bool ok = true;
            uint32_t nk = 0, nv = 0;                       // loads issued
            // keys and values that only one work unit reads are streamed through L2 with evict-first priority
            const bool stream_once = p.group == p.G;
            const uint64_t pol = l2_policy_evict_first();
            auto load_tile = [&](const Cursor& c, bool values, uint32_t slot) {
                const int lti = c.s.lt + c.i;
                const bool tree = lti >= c.s.nP;
                const int row0 = (tree ? lti - c.s.nP : lti) * kTile;
                const int bh_kv = c.s.b * p.Hkv + (c.s.h * p.G) / p.group;
                const uint32_t dst = smem_u32(ring) + slot * (uint32_t)kSlotBytes;
                // A tile with at most 64 rows in use (the ragged end of a prefix, a small tree) is fetched as a box of
                // 64 rows, so that fewer rows travel for nothing.  (Smaller boxes do not pay: a copy instruction has a
                // fixed cost in the copy unit, and a tile cut into 32-row boxes streams at half the rate.)  The rows
                // of the slot that are not fetched keep what an earlier tile left there: dead key rows are ignored,
                // value rows are finite (see the set-up).
                const int valid = min(kTile, (tree ? c.s.Nb : c.s.L) - row0);
                const bool half = loaded_rows(valid) < kTile;
                const CUtensorMap* map = half ? (values ? (tree ? &tm_vt64 : &tm_vc64) : (tree ? &tm_kt64 : &tm_kc64))
                                              : (values ? (tree ? &tm_vt : &tm_vc) : (tree ? &tm_kt : &tm_kc));
                mbar_expect_tx(&sm->slot_full[slot], half ? (uint32_t)kSlotBytes / 2u : (uint32_t)kSlotBytes);
                if (stream_once) {
                    tma_load_3d_hint(dst, map, &sm->slot_full[slot], 0, row0, bh_kv, pol);
                    tma_load_3d_hint(dst + kSlabBytes, map, &sm->slot_full[slot], 64, row0, bh_kv, pol);
                } else {
                    tma_load_3d(dst, map, &sm->slot_full[slot], 0, row0, bh_kv);
                    tma_load_3d(dst + kSlabBytes, map, &sm->slot_full[slot], 64, row0, bh_kv);
                }
            };
            auto advance = [&](Cursor& c) {
                c.t += 1;
                if (++c.i == c.cnt && c.t < t_end) open(c);
            };
            for (uint32_t n = 0; n <= total_n && ok; ++n) {
                if (n < total_n) {
                    if (ck.i == 0) {
                        // a new segment: its queries replace the previous segment's once that one's last S^T is done
                        if (n > 0) ok = mbar_wait(&sm->s_full[(n - 1u) & 1u], ((n - 1u) >> 1) & 1u, abort_flag, hdr, 1);
                        if (!ok) break;
                        const int bh = ck.s.b * p.H + ck.s.h;
                        mbar_expect_tx(&sm->q_full, (uint32_t)p.npadq * 256u);
                        if (p.G == 1) {
                            tma_load_3d(smem_u32(q_buf), &tm_q, &sm->q_full, 0, ck.s.q0, bh);
                            tma_load_3d(smem_u32(q_buf) + (uint32_t)p.npadq * 128u, &tm_q, &sm->q_full, 64, ck.s.q0, bh);
                        } else {
                            // grouped queries: a box of all G heads by npadq / G nodes lands node-major, i.e. as stacked
                            // queries q0, q0 + 1, ...
                            tma_load_4d(smem_u32(q_buf), &tm_q, &sm->q_full, 0, 0, ck.s.q0 >> p.g_shift, bh);
                            tma_load_4d(smem_u32(q_buf) + (uint32_t)p.npadq * 128u, &tm_q, &sm->q_full, 64, 0, ck.s.q0 >> p.g_shift, bh);
                        }
                    }
                    if (n >= 2) ok = mbar_wait(&sm->s_full[n & 1u], ((n - 2u) >> 1) & 1u, abort_flag, hdr, 2);
                    if (!ok) break;
                    load_tile(ck, false, n & 1u);
                    ++nk;
                    advance(ck);
                }
                if (n >= 1) {
                    const uint32_t m = n - 1u;
                    if (m >= 2) ok = mbar_wait(&sm->pv_done[m & 1u], ((m - 2u) >> 1) & 1u, abort_flag, hdr, 2);
                    if (!ok) break;
                    load_tile(cv, true, 2u + (m & 1u));
                    ++nv;
                    advance(cv);
                }
            }
            if (!ok) {
                // gave up: let the copies already issued land before the block exits
                for (int which = 0; which < 2; ++which) {
                    const uint32_t cnt_issued = which ? nv : nk;
                    for (uint32_t x = cnt_issued > 2 ? cnt_issued - 2 : 0; x < cnt_issued; ++x) {
                        void* bar = &sm->slot_full[2 * which + (x & 1u)];
                        const long long t0 = clock64();
                        while (!mbar_try_wait(bar, (x >> 1) & 1u) && clock64() - t0 < kSpinCycles / 8) {}
                    }
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // =========================================================== MMA issuer
        // The whole warp walks the loop (waits included) and one elected lane issues each tensor-core instruction
        // and each commit; shared-memory descriptors are built once and advanced by constants, so that the few
        // instructions between two MMAs do not pace the tensor pipe (small-N products take only 40-60 cycles).
        {
            long long t = t_begin;
            uint32_t g = 0, seg = 0;
            bool ok = true;
            const uint32_t ring_a = smem_u32(ring), q_a = smem_u32(q_buf), p_a = smem_u32(p_buf);
            const uint32_t idesc_l = instr_desc(16, 1, 0);
            const uint64_t dk0 = smem_desc(ring_a, 16, 1024, 2);                       // key slot 0, first 16 head dims
            const uint64_t dv0 = smem_desc(ring_a + 2 * kSlotBytes, kSlabBytes, 1024, 2);   // value slot 0, first 16 keys
            const uint64_t dq0 = smem_desc(q_a, 16, 1024, 2);
            const uint64_t dp0 = smem_desc(p_a, 128, 2048, 0);                         // P^T: B operand of O^T, A operand of l
            const uint64_t d1 = smem_desc(smem_u32(sm->ones), 128, 256, 0);
            const uint32_t q_slab = ((uint32_t)p.npadq * 128u) >> 4;                   // second 64 head dims of Q
            while (t < t_end && ok) {
                Segment s;
                locate<QB>(ix, p, t, s);
                const int cnt = (int)min((long long)(s.Tkv - s.lt), t_end - t);
                const int npad = (s.Nq + 15) & ~15;
                const uint32_t idesc_s = instr_desc(npad, 0, 0), idesc_pv = instr_desc(npad, 1, 1);
                const bool two = NCH == 10 && s.Nq > 128;
                ok = mbar_wait(&sm->q_full, seg & 1u, abort_flag, hdr, 3);
                for (int i = 0; i <= cnt && ok; ++i) {
                    if (i < cnt) {
                        const uint32_t gi = g + (uint32_t)i, sb = gi & 1u;
                        ok = mbar_wait(&sm->slot_full[sb], (gi >> 1) & 1u, abort_flag, hdr, 4);
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t da = dk0 + sb * (uint32_t)(kSlotBytes >> 4);
                        const uint32_t d_s = tmem + (sb ? kColS1 : 0);
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            // 16 of the 128 head dims per MMA: slab k/4, 32-byte step inside the swizzled row
                            tc_mma_elect(d_s, da + (uint32_t)((k >> 2) * (kSlabBytes >> 4) + (k & 3) * 2),
                                         dq0 + ((k >> 2) * q_slab + (uint32_t)(k & 3) * 2u), idesc_s, k > 0);
                        }
                        tc_commit_elect(&sm->s_full[sb]);
                        if (t + i + 1 == t_end) tc_commit_elect(&sm->s_last);
                    }
                    if (i >= 1) {
                        const uint32_t gj = g + (uint32_t)(i - 1), vb = gj & 1u;
                        ok = mbar_wait(&sm->slot_full[2u + vb], (gj >> 1) & 1u, abort_flag, hdr, 5);
                        if (!ok) break;
                        {
                            // Value rows past the end of the prefix (or past the active tree nodes) may hold anything,
                            // NaN patterns included, and 0 * NaN is NaN: they are cleared here, by the warp that waits
                            // for the tile anyway (the softmax warps would have to wait for a tile they do not need
                            // yet).  Rows the copy did not find in the tensor arrived as zeros.  Whole rows: the
                            // 128-byte swizzle only permutes inside a row.
                            const int ltv = s.lt + i - 1;
                            const bool tree_v = ltv >= s.nP;
                            const int row0_v = (tree_v ? ltv - s.nP : ltv) * kTile;
                            const int valid_v = min(kTile, (tree_v ? s.Nb : s.L) - row0_v);
                            // rows that were fetched and exist in the tensor
                            const int have_v = min(loaded_rows(valid_v), (tree_v ? p.N : p.L_max) - row0_v);
                            if (valid_v < have_v) {
                                unsigned char* v0 = ring + (size_t)(2u + vb) * kSlotBytes;
                                for (int c = valid_v * 8 + lane; c < have_v * 8; c += 32) {
                                    *reinterpret_cast<uint4*>(v0 + (size_t)c * 16) = make_uint4(0, 0, 0, 0);
                                    *reinterpret_cast<uint4*>(v0 + kSlabBytes + (size_t)c * 16) = make_uint4(0, 0, 0, 0);
                                }
                                fence_async_smem();
                                __syncwarp();
                            }
                        }
                        ok = mbar_wait(&sm->p_full, gj & 1u, abort_flag, hdr, 6);
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t da = dv0 + vb * (uint32_t)(kSlotBytes >> 4);
                        const uint32_t first = (i == 1) ? 0u : 1u;      // the segment's first product overwrites
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            // 16 keys per MMA.  V^T: 8-key groups 1 KB apart; P^T: 8-key groups 128 B apart.
                            tc_mma_elect(tmem + kColO, da + (uint32_t)(k * (2048 >> 4)), dp0 + (uint32_t)(k * (256 >> 4)), idesc_pv,
                                         first | (uint32_t)(k > 0));
                        }
                        // Row sums: l[query][.] += P[query][key] * ones[key][.], P^T read as the A operand (queries on
                        // the accumulator's lanes); queries 128.. take a second product into their own columns.
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            tc_mma_elect(tmem + kColL, dp0 + (uint32_t)(k * (256 >> 4)), d1, idesc_l, first | (uint32_t)(k > 0));
                        if (two) {
#pragma unroll
                            for (int k = 0; k < 8; ++k)
                                tc_mma_elect(tmem + kColL2, dp0 + (uint32_t)((16 * 2048 + k * 256) >> 4), d1, idesc_l,
                                             first | (uint32_t)(k > 0));
                        }
                        tc_commit_elect(&sm->pv_done[vb]);
                    }
                }
                g += (uint32_t)cnt;
                ++seg;
                t += cnt;
            }
            // all MMAs issued by this warp must have finished before tensor memory is released
            tc_commit_elect(&sm->drain);
            {
                const long long t0 = clock64();
                while (!mbar_try_wait(&sm->drain, 0) && clock64() - t0 < kSpinCycles) {}
            }
        }
    } else if (warp < kProducerWarp) {
        // =========================================================== softmax / mask / epilogue
        const int wg = warp >> 2, wq = warp & 3;
        const int r = tid & 127;                       // key row of a tile = TMEM lane
        const int bar_id = 1 + wg;
        float* const mref = sm->m_ref[wg];
        float* const alph = sm->alpha[wg];
        // dmask[t] = set of stacked queries that may see tree key t: the ancestor bitsets transposed (staged through
        // the P^T buffer, which is free until the first tile is finished).
        {
            unsigned long long* anc_s = reinterpret_cast<unsigned long long*>(p_buf);
            const int n_words = p.N * p.words;                   // at most 192 * 3 words = 4.5 KB
            for (int i = tid; i < n_words; i += 128 * kGroups) anc_s[i] = p.anc[i];
            asm volatile("bar.sync %0, %1;" ::"n"(kGroups + 1), "n"(128 * kGroups) : "memory");
            const int NQ = p.N * p.G;                            // stacked queries: query j belongs to node j / G
            const int n_kb = (p.N + 31) >> 5;                    // blocks of 32 tree keys
            const uint32_t* anc32 = reinterpret_cast<const uint32_t*>(anc_s);
            // a warp transposes one 32 x 32 block of bits at a time: lane i holds the keys 32 kb .. 32 kb + 31 that
            // stacked query 32 c + i may see; the ballot over bit j is the set of those queries that see key 32 kb + j
            for (int pair = warp; pair < 6 * n_kb; pair += 4 * kGroups) {
                const int c = pair / n_kb, kb = pair - c * n_kb;
                const int qi = 32 * c + lane;
                const uint32_t w = qi < NQ ? anc32[(size_t)(qi >> p.g_shift) * p.words * 2 + kb] : 0u;
                uint32_t mine = 0;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const uint32_t seen_by = __ballot_sync(0xffffffffu, (w >> j) & 1u);
                    if (lane == j) mine = seen_by;
                }
                const int t = 32 * kb + lane;
                if (t < p.N) reinterpret_cast<uint32_t*>(&sm->dmask[t][0])[c] = mine;
            }
            asm volatile("bar.sync %0, %1;" ::"n"(kGroups + 1), "n"(128 * kGroups) : "memory");
        }
        const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
        long long t = t_begin;
        uint32_t g = 0;
        bool failed = false;
        bool ticket_owed = false;                      // the block's first segment continues another block's work item
        while (t < t_end) {
            Segment s;
            locate<QB>(ix, p, t, s);
            const int cnt = (int)min((long long)(s.Tkv - s.lt), t_end - t);
            const int bh = s.b * p.H + s.h;
            if (t == t_begin) ticket_owed = s.lt > 0;
            // the groups split the segment's 8-column groups as evenly as possible
            const int ng8 = (s.Nq + 7) >> 3;
            const int base = ng8 / kGroups, rem = ng8 % kGroups;
            const int g0 = wg * base + min(wg, rem);
            const int ncg = base + (wg < rem ? 1 : 0);           // 8-column groups of this thread in this segment
            const int col0 = g0 * 8;
            // Row sums: lane q of the first set of row-sum columns holds the sum of query q, lane q - 128 of the second
            // set that of query q >= 128; the 16 columns of a set are identical copies, and group wg only ever
            // touches copy wg (a rescale is a read-modify-write that must not race with another group's).  A warp's
            // 32 lanes hold queries of one set only, so the set is chosen per warp (tcgen05.ld/st are warp-wide).
            const bool set2 = (128 + 32 * wq < col0 + 8 * ncg) && (128 + 32 * wq + 32 > col0);
            const int oq_c = set2 ? 128 + r : r;
            const int oq = (oq_c >= col0 && oq_c < col0 + 8 * ncg) ? oq_c : -1;   // this thread's query, if of this group
            const uint32_t l_addr = tmem + lane_addr + (set2 ? kColL2 : kColL) + wg;
            if (r < ncg * 8) mref[r] = -INFINITY;
            if (group_sync_any(bar_id, failed)) { failed = true; break; }

            for (int i = 0; i < cnt; ++i) {
                const uint32_t gi = g + (uint32_t)i, sb = gi & 1u;
                const int lti = s.lt + i;
                const bool tree = lti >= s.nP;
                const int row0 = (tree ? lti - s.nP : lti) * kTile;
                const int valid = min(kTile, (tree ? s.Nb : s.L) - row0);
                const bool full_tile = !tree && valid == kTile;   // every key visible to every query: no masking
                // queries that may see this thread's key (bit n), shifted to this thread's first column
                unsigned long long cm = 0;
                if (!full_tile && r < valid) {
                    const int nrem = s.Nq - col0;
                    cm = nrem >= 64 ? ~0ull : (nrem > 0 ? ((1ull << nrem) - 1ull) : 0ull);
                    if (tree) cm &= bits_from(sm->dmask[row0 + r], s.q0 + col0);
                }
                if (!mbar_wait(&sm->s_full[sb], (gi >> 1) & 1u, abort_flag, hdr, 7)) failed = true;
                tc_fence_after();
                const uint32_t s_addr = tmem + lane_addr + (sb ? kColS1 : 0) + col0;

                // ---- the sweep: scores of this thread's columns, shifted, checked, exponentiated, packed; tensor memory
                // is read SB column groups per round trip (what the 128 registers of a 16-warp block allow).  Prefix
                // tiles take the plain sweep: every query sees every key, and a key row past the end of a ragged last
                // tile is this thread's own row, cleared afterwards.  Tree tiles take the masked sweep, which clears
                // single elements: the packed probabilities are ANDed with masks grown from the visibility bits, and
                // the largest visible probability (bf16 bit patterns of positive numbers order like the numbers)
                // stands in for the largest shifted score.
                constexpr int SB = 2;
                uint32_t pk[CPT][4];
                float dmax = -INFINITY;
                auto make_probs = [&](auto masked_tag) {
                    constexpr bool MASKED = decltype(masked_tag)::value;
                    uint32_t pmax = 0;
#pragma unroll
                    for (int j0 = 0; j0 < CPT; j0 += SB) {
                        if (j0 < ncg) {
                            float y[SB][8];
#pragma unroll
                            for (int jj = 0; jj < SB; ++jj)
                                if (j0 + jj < CPT && j0 + jj < ncg) tc_ld8(s_addr + 8 * (j0 + jj), y[jj]);
                            tc_wait_ld();
#pragma unroll
                            for (int jj = 0; jj < SB; ++jj) {
                                const int j = j0 + jj;
                                if (j < CPT && j < ncg) {
                                    const float4 m0 = *reinterpret_cast<const float4*>(&mref[8 * j]);
                                    const float4 m1 = *reinterpret_cast<const float4*>(&mref[8 * j + 4]);
                                    const float mr[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
                                    float yy[8];
#pragma unroll
                                    for (int k = 0; k < 8; ++k) yy[k] = fmaf(y[jj][k], p.scale_log2, -mr[k]);
                                    if (!MASKED)
                                        dmax = fmaxf(dmax, fmaxf(fmaxf(fmaxf(yy[0], yy[1]), fmaxf(yy[2], yy[3])),
                                                                 fmaxf(fmaxf(yy[4], yy[5]), fmaxf(yy[6], yy[7]))));
#pragma unroll
                                    for (int k = 0; k < 8; k += 2) {
                                        __nv_bfloat162 h2 = __floats2bfloat162_rn(ex2_approx(yy[k]), ex2_approx(yy[k + 1]));
                                        pk[j][k >> 1] = *reinterpret_cast<uint32_t*>(&h2);
                                    }
                                    if (MASKED) {
                                        // visibility bit k -> top bit of byte k (a multiply that spreads four bits), then
                                        // a byte permute that replicates those top bits over the halves of a word
                                        const uint32_t bits = (uint32_t)(cm >> (8 * j)) & 0xFFu;
                                        const uint32_t lo4 = (bits & 0xFu) * 0x10204080u, hi4 = (bits >> 4) * 0x10204080u;
                                        pk[j][0] &= prmt(lo4, 0u, 0x9988u);
                                        pk[j][1] &= prmt(lo4, 0u, 0xBBAAu);
                                        pk[j][2] &= prmt(hi4, 0u, 0x9988u);
                                        pk[j][3] &= prmt(hi4, 0u, 0xBBAAu);
                                        pmax = max_u16x2(pmax, max_u16x2(max_u16x2(pk[j][0], pk[j][1]), max_u16x2(pk[j][2], pk[j][3])));
                                    }
                                }
                            }
                        }
                    }
                    // 0x4380 is 2^kLazyTau = 256 in bf16; NaN patterns are above it too
                    if (MASKED) dmax = max(pmax & 0xFFFFu, pmax >> 16) > 0x4380u ? INFINITY : -INFINITY;
                };
                if (i == 0 && full_tile) {
                    // reference of a new segment: the scores of one key of the tile (see the file header).  The four
                    // warps of the group share the column groups; warp wq samples key 32 wq, the row its lane 0 holds.
#pragma unroll
                    for (int j = 0; j < CPT; ++j) {
                        if (j < ncg && (j & 3) == wq) {
                            float v[8];
                            tc_ld8(s_addr + 8 * j, v);
                            tc_wait_ld();
                            if (lane == 0) {
#pragma unroll
                                for (int k = 0; k < 8; ++k) mref[8 * j + k] = v[k] * p.scale_log2;
                            }
                        }
                    }
                    group_sync_any(bar_id, false);
                }
                auto sweep = [&]() {
                    if (!tree) {
                        make_probs(std::false_type{});
                        if (r >= valid) {                      // a key row past the end of the prefix: seen by no query
                            dmax = -INFINITY;
#pragma unroll
                            for (int j = 0; j < CPT; ++j) pk[j][0] = pk[j][1] = pk[j][2] = pk[j][3] = 0u;
                        }
                    } else {
                        make_probs(std::true_type{});
                    }
                };
                sweep();
                // one vote per group: does any score exceed its reference by more than the lazy threshold?
                if (group_sync_any(bar_id, dmax > kLazyTau || failed)) {
                    if (*(volatile int*)&sm->abort_flag) { failed = true; break; }
                    // ---- slow path: exact per-query maxima of this tile, new reference, rescale what was accumulated
#pragma unroll
                    for (int j = 0; j < CPT; ++j) {
                        if (j < ncg) {
                            float v[8];
                            tc_ld8(s_addr + 8 * j, v);
                            tc_wait_ld();
                            const uint32_t bits = (uint32_t)(cm >> (8 * j)) & 0xFFu;
                            float mine = -INFINITY;
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                const float x = (full_tile || ((bits >> k) & 1u)) ? v[k] * p.scale_log2 : -INFINITY;
                                const float mx = warp_max_f32(x);
                                if (lane == k) mine = mx;
                            }
                            if (lane < 8) sm->wred[wg][wq][8 * j + lane] = mine;
                        }
                    }
                    group_sync_any(bar_id, false);
                    bool need = false;
                    if (r < ncg * 8) {
                        const float tm = fmaxf(fmaxf(sm->wred[wg][0][r], sm->wred[wg][1][r]),
                                               fmaxf(sm->wred[wg][2][r], sm->wred[wg][3][r]));
                        const float mo = mref[r];
                        float a = 1.f;
                        if (tm > mo) {
                            a = (mo == -INFINITY) ? 0.f : exp2f(mo - tm);
                            mref[r] = tm;
                            need = (i > 0) && (mo != -INFINITY);
                        }
                        alph[r] = a;
                    }
                    const bool rescale = group_sync_any(bar_id, need);
                    if (gi > 0 && !mbar_wait(&sm->pv_done[(gi - 1u) & 1u], ((gi - 1u) >> 1) & 1u, abort_flag, hdr, 8)) failed = true;
                    if (rescale) {
                        tc_fence_after();
                        {                                // the row sum accumulated so far belongs to the old reference
                            const float lp = tc_ld1(l_addr);
                            tc_wait_ld();
                            tc_st1(l_addr, oq >= 0 ? lp * alph[oq - col0] : lp);
                        }
#pragma unroll
                        for (int j = 0; j < CPT; ++j) {
                            if (j < ncg) {
                                float o[8];
                                tc_ld8(tmem + lane_addr + kColO + col0 + 8 * j, o);
                                tc_wait_ld();
#pragma unroll
                                for (int k = 0; k < 8; ++k) o[k] *= alph[8 * j + k];
                                tc_st8(tmem + lane_addr + kColO + col0 + 8 * j, o);
                            }
                        }
                        tc_wait_st();
                    }
                    dmax = -INFINITY;
                    sweep();
                }

                // P buffer must no longer be read by the previous tile's MMA; this wait also keeps every thread
                // within one phase of the p_full barrier
                if (gi > 0 && !mbar_wait(&sm->pv_done[(gi - 1u) & 1u], ((gi - 1u) >> 1) & 1u, abort_flag, hdr, 8)) failed = true;
#pragma unroll
                for (int j = 0; j < CPT; ++j)
                    if (j < ncg)
                        *reinterpret_cast<uint4*>(p_buf + (size_t)(g0 + j) * 2048 + (size_t)r * 16) =
                            make_uint4(pk[j][0], pk[j][1], pk[j][2], pk[j][3]);
                // every thread makes its own P^T stores visible to the tensor cores' proxy; then one arrival per warp (384
                // arrivals on one shared-memory word would queue up behind one another)
                fence_async_smem();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->p_full);
            }
            if (group_sync_any(bar_id, failed)) { failed = true; break; }

            // ---- epilogue of the segment: each group finishes its own query columns.  A segment that holds a whole work
            // item is normalised and written out.  A piece of a split item that does not start the item is written to
            // the workspace unnormalised and announced with a ticket.  The piece that starts a split item is always a
            // block's last segment: it stays in tensor memory and the whole block merges the other pieces into it (see
            // the end of the kernel), so there is nothing to do here.
            const uint32_t glast = g + (uint32_t)cnt - 1u;
            const bool full = (cnt == s.Tkv);
            if (!full && s.lt == 0) break;
            const int slot_id = 2 * cta + (t > t_begin ? 1 : 0);
            if (!mbar_wait(&sm->pv_done[glast & 1u], (glast >> 1) & 1u, abort_flag, hdr, 10)) failed = true;
            tc_fence_after();
            const float l = tc_ld1(l_addr);
            tc_wait_ld();
            if (oq >= 0) {
                // the row sum of query oq sits in this thread's lane: hand it to the threads that finish its column
                if (full) {
                    alph[oq - col0] = l > 0.f ? 1.f / l : 0.f;
                } else {
                    alph[oq - col0] = l;               // kept for the merge below
                    p.part_ml[((size_t)slot_id * 2 + 0) * kMaxQ + oq] = mref[oq - col0];
                    p.part_ml[((size_t)slot_id * 2 + 1) * kMaxQ + oq] = l;
                }
            }
            group_sync_any(bar_id, false);
            // O^T rows of this thread, one column group per tensor-memory round trip (registers)
            constexpr int EB = 1;
#pragma unroll
            for (int j0 = 0; j0 < CPT; j0 += EB) {
                if (j0 < ncg) {
                    float o[EB][8];
#pragma unroll
                    for (int jj = 0; jj < EB; ++jj)
                        if (j0 + jj < CPT && j0 + jj < ncg) tc_ld8(tmem + lane_addr + kColO + col0 + 8 * (j0 + jj), o[jj]);
                    tc_wait_ld();
#pragma unroll
                    for (int jj = 0; jj < EB; ++jj) {
                        const int j = j0 + jj;
                        if (j < CPT && j < ncg) {
                            if (full) {
                                // Thread r holds head dim r of eight queries.  An 8 x 8 transpose inside every group of
                                // eight lanes (three butterfly stages) leaves lane 8a + k with eight consecutive head
                                // dims of query k: one 16-byte store per thread instead of eight 2-byte ones.
                                float v[8];
#pragma unroll
                                for (int k = 0; k < 8; ++k) v[k] = o[jj][k] * alph[8 * j + k];
#pragma unroll
                                for (int m = 4; m > 0; m >>= 1) {
                                    const bool up = lane & m;
#pragma unroll
                                    for (int x = 0; x < 8; ++x) {
                                        if (x & m) continue;
                                        const float send = up ? v[x] : v[x | m];
                                        const float got = __shfl_xor_sync(0xffffffffu, send, m);
                                        if (up) v[x] = got; else v[x | m] = got;
                                    }
                                }
                                const int n = col0 + 8 * j + (lane & 7);
                                if (n < s.Nq) {
                                    uint4 w;
                                    __nv_bfloat162 h;
                                    h = __floats2bfloat162_rn(v[0], v[1]); w.x = *reinterpret_cast<uint32_t*>(&h);
                                    h = __floats2bfloat162_rn(v[2], v[3]); w.y = *reinterpret_cast<uint32_t*>(&h);
                                    h = __floats2bfloat162_rn(v[4], v[5]); w.z = *reinterpret_cast<uint32_t*>(&h);
                                    h = __floats2bfloat162_rn(v[6], v[7]); w.w = *reinterpret_cast<uint32_t*>(&h);
                                    const int jq = s.q0 + n;          // stacked query: head jq % G of the group, node jq / G
                                    *reinterpret_cast<uint4*>(p.out + (((size_t)bh * p.G + (jq & (p.G - 1))) * p.N + (jq >> p.g_shift)) * 128 +
                                                              32 * wq + (lane & 24)) = w;
                                }
                            } else {
#pragma unroll
                                for (int k = 0; k < 8; ++k) {
                                    const int n = col0 + 8 * j + k;
                                    if (n < s.Nq) p.part_o[((size_t)slot_id * kMaxQ + n) * 128 + r] = o[jj][k];
                                }
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            if (!full) {
                // The partial is complete.  Making it visible device-wide takes a microsecond or two under load, so
                // the fence and the ticket the merging block waits for are left to the last service warp: the
                // arrival orders this thread's stores before that warp's fence.
                asm volatile("bar.arrive %0, %1;" ::"n"(kGroups + 4), "n"(128 * kGroups + 32) : "memory");
                ticket_owed = false;
            }
            group_sync_any(bar_id, false);
            g += (uint32_t)cnt;
            t += cnt;
        }
        // gave up before the partial was written: the service warp must not wait for this thread
        if (ticket_owed) asm volatile("bar.arrive %0, %1;" ::"n"(kGroups + 4), "n"(128 * kGroups + 32) : "memory");
    }

    // =========================================================== merge of a split work item
    // If this block's last segment starts a work item that continues in later blocks, the block folds the other
    // pieces, which those blocks produced as the first thing they did, into its own piece, still in tensor memory:
    //     m = max(m_a, m_b),  l = l_a 2^(m_a - m) + l_b 2^(m_b - m),  O = O_a 2^(m_a - m) + O_b 2^(m_b - m),  o = O / l.
    // Thread r holds head dim r of every query.  Under a saturated memory system a dependent trip to the workspace
    // costs 1.5-2 us, so there is one per piece: the piece's rows and its (m, l) are brought into the (now idle)
    // key/value ring with two bulk copies.  The tickets that say the pieces are complete are polled, at leisure, by
    // a warp that has nothing else to do, long before they are needed.  The code lives after the roles' branches,
    // away from the softmax warps' tile loop, so that its registers are its own.
    if (warp >= kProducerWarp) {
        if (warp == kMmaWarp + 1) {
            if (lane == 0) {
                Segment sp;
                locate<QB>(ix, p, t_end - 1, sp);
                const long long t0 = t_end - 1 - sp.lt, t1 = t0 + sp.Tkv;
                int np1 = 0;
                if (t1 > t_end && t0 >= t_begin) {
                    np1 = min(block_of_tile<QB>(ix, p, t1 - 1, G, total_w) - cta, kMaxParts - 1);
                    // one counter per softmax group of the writing blocks; np1 arrivals each
                    int* counter = p.counters + ((size_t)(sp.b * p.H + sp.h) * 2 + sp.qb) * 4;
                    const long long t_start = clock64();
                    for (int gq = 0; gq < kGroups; ++gq) {
                        while (*(volatile int*)(counter + gq) < np1) {
                            __nanosleep(500);
                            if (*(volatile int*)abort_flag || clock64() - t_start > kSpinCycles) {
                                *(volatile int*)abort_flag = 1;
                                hdr->detail = 14;
                                hdr->status = MCSD_ERR_TIMEOUT;
                                break;
                            }
                        }
                        *(volatile int*)(counter + gq) = 0;       // ready for the next launch
                    }
                    __threadfence();                              // acquire: the pieces' partials are visible
                }
                // The first piece is fetched as soon as there is room: once the block's last S^T has finished, the
                // two key slots (64 KB) and the Q buffer are free, one and a half tiles before the block is done.
                int prefetched = 0;
                const uint32_t o_bytes = (uint32_t)((sp.Nq + 7) >> 3) * 4096u;
                if (np1 > 0 && o_bytes <= 2u * kSlotBytes && !*(volatile int*)abort_flag &&
                    mbar_wait(&sm->s_last, 0, abort_flag, hdr, 15)) {
                    const size_t slot = (size_t)(2 * (cta + 1));
                    asm volatile("fence.proxy.async;" ::: "memory");
                    mbar_expect_tx(&sm->merge_bar, o_bytes + 2u * kMaxQ * 4u);
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(smem_u32(ring)), "l"(p.part_o + slot * kMaxQ * 128), "r"(o_bytes), "r"(smem_u32(&sm->merge_bar)) : "memory");
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(smem_u32(q_buf)), "l"(p.part_ml + slot * 2 * kMaxQ), "r"(2u * kMaxQ * 4u), "r"(smem_u32(&sm->merge_bar)) : "memory");
                    prefetched = 1;
                }
                sm->merge_prefetched = prefetched;
                sm->merge_np1 = np1;
                sm->merge_item = sp;
            }
            __syncwarp();
        }
        if (warp == kMmaWarp + 2) {
            // ticket of a partial: if this block's first segment continues a work item, the softmax warps arrive here
            // once its partial is written; this warp makes it visible and takes one ticket per softmax group
            Segment sf;
            locate<QB>(ix, p, t_begin, sf);
            if (sf.lt > 0) {
                asm volatile("bar.sync %0, %1;" ::"n"(kGroups + 4), "n"(128 * kGroups + 32) : "memory");
                __threadfence();
                if (lane < kGroups && !*(volatile int*)abort_flag)
                    atomicAdd(p.counters + ((size_t)(sf.b * p.H + sf.h) * 2 + sf.qb) * 4 + lane, 1);
            }
        }
    }
    // Every role is done with its loop (a hardware barrier: the warps that get here early sleep instead of taking issue
    // slots from the softmax warps).  The merge itself is shared by all sixteen warps: warp w reaches tensor-memory
    // lanes 32 (w % 4) .., i.e. head dims, and takes every fourth 8-column group, starting with group w / 4.
    tc_fence_before();
    __syncthreads();
    {
        const int np1 = sm->merge_np1;
        if (np1 > 0) {
            const int r = 32 * (warp & 3) + lane;                // tensor-memory lane = head dim
            const int part = warp >> 2;                          // 0..3: which column groups
            const Segment sp = sm->merge_item;
            const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
            const int bh = sp.b * p.H + sp.h;
            float* const l_run = &sm->wred[0][0][0];             // [160] running normaliser, at the end 1 / l
            float* const m_run = l_run + kMaxQ;                  // [160] running reference
            float* const w_a = m_run + kMaxQ;                    // [160] weight of what has been combined so far
            float* const w_b = w_a + kMaxQ;                      // [160] weight of the piece being added
            static_assert(4 * kMaxQ <= kGroups * 4 * 64, "the merge scratch must fit the per-warp reduction scratch");
            const float* stage_o = reinterpret_cast<const float*>(ring);                     // [<= 160][128]
            const float* stage_ml = reinterpret_cast<const float*>(q_buf);                   // [2][160]
            // column -> (softmax group, index within the group), as the softmax warps split this segment
            const int ng8 = (sp.Nq + 7) >> 3, base = ng8 / kGroups, rem = ng8 % kGroups;
            auto group_of = [&](int q, int& rel) {
                const int g8 = q >> 3;
                int gidx = 0;
#pragma unroll
                for (int x = 1; x < kGroups; ++x) gidx += (g8 >= x * base + min(x, rem)) ? 1 : 0;
                rel = q - 8 * (gidx * base + min(gidx, rem));
                return gidx;
            };
            // All of this block's tensor-core work has finished (the MMA warp waited for its last commit before the
            // barrier above).
            tc_fence_after();
            // this block's own row sums and references: lane q of the first set of row-sum columns holds query q, lane
            // q - 128 of the second set query q; the copy kept current is number (group of q)
            if (part == 3) {
                float c1[4], c2[4];
                tc_ld4(tmem + lane_addr + kColL, c1);
                tc_ld4(tmem + lane_addr + kColL2, c2);
                tc_wait_ld();
                int rel;
                if (r < sp.Nq) { const int gq = group_of(r, rel); l_run[r] = gq == 0 ? c1[0] : gq == 1 ? c1[1] : c1[2]; m_run[r] = sm->m_ref[gq][rel]; }
                if (128 + r < sp.Nq) { const int gq = group_of(128 + r, rel); l_run[128 + r] = gq == 0 ? c2[0] : gq == 1 ? c2[1] : c2[2]; m_run[128 + r] = sm->m_ref[gq][rel]; }
            }
            for (int i = 1; i <= np1; ++i) {
                const size_t slot = (size_t)(2 * (cta + i));       // the piece is that block's first segment
                // staging area and weights are free, l_run and m_run written; all threads agree on giving up
                if (!__syncthreads_and(!*(volatile int*)abort_flag)) break;
                if (tid == 0 && !(i == 1 && sm->merge_prefetched)) {
                    const uint32_t o_bytes = (uint32_t)ng8 * 4096u, ml_bytes = 2u * kMaxQ * 4u;
                    asm volatile("fence.proxy.async;" ::: "memory");
                    mbar_expect_tx(&sm->merge_bar, o_bytes + ml_bytes);
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(smem_u32(stage_o)), "l"(p.part_o + slot * kMaxQ * 128), "r"(o_bytes), "r"(smem_u32(&sm->merge_bar)) : "memory");
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(smem_u32(stage_ml)), "l"(p.part_ml + slot * 2 * kMaxQ), "r"(ml_bytes), "r"(smem_u32(&sm->merge_bar)) : "memory");
                }
                const bool ok = mbar_wait(&sm->merge_bar, (uint32_t)(i - 1) & 1u, abort_flag, hdr, 13);
                const bool last = i == np1;
                if (tid < sp.Nq) {
                    const int q = tid;
                    const float ma = m_run[q], mb = stage_ml[q], lb = stage_ml[kMaxQ + q];
                    const float mn = fmaxf(ma, mb);
                    const float wa = (mn == -INFINITY || ma == -INFINITY) ? 0.f : exp2f(ma - mn);
                    const float wb = (mn == -INFINITY || mb == -INFINITY) ? 0.f : exp2f(mb - mn);
                    const float ln = l_run[q] * wa + lb * wb;
                    m_run[q] = mn;
                    w_a[q] = wa;
                    w_b[q] = wb;
                    l_run[q] = last ? (ln > 0.f ? 1.f / ln : 0.f) : ln;
                }
                if (!__syncthreads_and(ok)) break;
#pragma unroll 1
                for (int j = part; j < ng8; j += 4) {
                    float acc[8];
                    tc_ld8(tmem + lane_addr + kColO + 8 * j, acc);
                    tc_wait_ld();
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int q = 8 * j + k;
                        acc[k] = fmaf(stage_o[(size_t)q * 128 + r], w_b[q], acc[k] * w_a[q]);
                    }
                    if (last) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const int q = 8 * j + k;
                            if (q < sp.Nq) {
                                const int jq = sp.q0 + q;   // stacked query: head jq % G of the group, node jq / G
                                p.out[(((size_t)bh * p.G + (jq & (p.G - 1))) * p.N + (jq >> p.g_shift)) * 128 + r] =
                                    __float2bfloat16_rn(acc[k] * l_run[q]);
                            }
                        }
                    } else {
                        tc_st8(tmem + lane_addr + kColO + 8 * j, acc);
                    }
                }
                if (!last) tc_wait_st();
            }
        }
    }

    // ---- tear-down
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ------------------------------------------------------------------ self-test of the bounded waits
// One block waits, with the kernel's own wait routine and a short limit, on a barrier that nothing ever completes:
// the wait must give up, raise the flag the other roles watch, leave MCSD_ERR_TIMEOUT and the wait's code in the
// workspace header, and the block must exit normally.  A second warp that starts its wait afterwards must give up
// at once because of the flag.
__global__ void bounded_wait_selftest_kernel(WorkspaceHeader* header, long long limit_cycles, int where) {
    __shared__ unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool ok = true;
    if (threadIdx.x < 32) ok = mbar_wait_slow(&bar, 0, &abort_flag, header, where, limit_cycles);
    __syncthreads();
    if (threadIdx.x >= 32) ok = mbar_wait_slow(&bar, 0, &abort_flag, header, where + 100, 1LL << 40);   // sees the flag: no long wait
    if (ok) header->detail = -1;                               // must not happen
}

int tc_bounded_wait_selftest(WorkspaceHeader* header, long long limit_cycles, int where, cudaStream_t stream) {
    bounded_wait_selftest_kernel<<<1, 64, 0, stream>>>(header, limit_cycles, where);
    MCSD_CUDA_CHECK(cudaGetLastError());
    count_launches(1);
    return MCSD_OK;
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    });
    return fn;
}

// Tensor maps depend only on (base pointer, rows, B*H, box rows).  A decode loop calls with the same few
// buffers every step, so the encoded maps are kept in a small per-thread table (round-robin replacement).
struct MapKey {
    const void* base;
    int rows, bh, box_rows, group;
};
constexpr int kMapCacheSize = 256;
struct MapCache {
    MapKey key[kMapCacheSize];
    CUtensorMap map[kMapCacheSize];
    int used = 0, next = 0;
};
static thread_local MapCache g_map_cache;

static bool encode_map(CUtensorMap* map, const void* base, int rows, int bh, int box_rows, int group);

// group == 1: [BH][rows][128] bf16 tensor, boxes of box_rows x 64 columns, 128-byte swizzle, zero fill outside.
// group  > 1: the queries of a grouped-query target, [BH][group][rows][128]: dimensions (column, head of the
//             group, row, BH) so that a box of all heads by box_rows / group rows lands row-major in shared memory.
static bool make_map(CUtensorMap* map, const void* base, int rows, int bh, int box_rows, int group = 1) {
    MapCache& c = g_map_cache;
    for (int i = 0; i < c.used; ++i) {
        const MapKey& k = c.key[i];
        if (k.base == base && k.rows == rows && k.bh == bh && k.box_rows == box_rows && k.group == group) {
            *map = c.map[i];
            return true;
        }
    }
    if (!encode_map(map, base, rows, bh, box_rows, group)) return false;
    const int slot = c.used < kMapCacheSize ? c.used++ : (c.next = (c.next + 1) % kMapCacheSize);
    c.key[slot] = MapKey{base, rows, bh, box_rows, group};
    c.map[slot] = *map;
    return true;
}

static bool encode_map(CUtensorMap* map, const void* base, int rows, int bh, int box_rows, int group) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    if (group > 1) {
        cuuint64_t dims[4] = {128, (cuuint64_t)group, (cuuint64_t)rows, (cuuint64_t)bh};
        cuuint64_t strides[3] = {(cuuint64_t)rows * 256, 256, (cuuint64_t)group * rows * 256};
        cuuint32_t box[4] = {64, (cuuint32_t)group, (cuuint32_t)(box_rows / group), 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    }
    cuuint64_t dims[3] = {128, (cuuint64_t)rows, (cuuint64_t)bh};
    cuuint64_t strides[2] = {256, (cuuint64_t)rows * 256};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Padded query columns of a launch in 16-column chunks: 3, 4, 7, 8 or 10 (10 = 160 queries in one pass; trees with
// more stacked queries are cut into blocks of 160).
static int chunks_for(int nq) {
    const int nch = ((nq < kMaxQ ? nq : kMaxQ) + 15) / 16;
    return nch <= 3 ? 3 : nch <= 4 ? 4 : nch <= 7 ? 7 : nch <= 8 ? 8 : 10;
}

// Query heads of one key/value group stacked into one work unit: the largest of 8, 4, 2, 1 that divides the group
// and keeps the stacked queries within one query block (a second block would stream the keys again, which is what
// a second unit does as well, with narrower tiles).
static int tc_stack_for(int G, int N) {
    for (int s = 8; s > 1; s >>= 1)
        if (G % s == 0 && s * N <= kMaxQ) return s;
    return 1;
}

// Shapes the tensor-core kernel takes.  B <= 256 (per-sequence tables in shared memory); the per-sequence prefix sums
// of tiles and cost units are 32-bit, so the largest launch is bounded so that they cannot wrap (a sequence of L_max
// keys and 192 nodes costs at most 2 * (tiles + 4) * 64 units per head): B * (L_max / 128 + 4) < 2^23, i.e. a
// 4-million-token prefix at B = 256 and a 500-million-token one at B = 2.
bool tc_shape_supported(int B, int H, int G, int N, int D, int L_max, int dtype) {
    if (dtype != MCSD_BF16 || D != 128) return false;
    if (!(G >= 1 && H % G == 0 && N >= 1 && N <= MCSD_MAX_NODES && B >= 1 && B <= kMaxBatchTc && L_max >= 0)) return false;
    const long long tiles = (long long)L_max / kTile + 4;
    return (long long)B * tiles * 2 * 64 < (1LL << 30);
}

// The kernel's plan evaluated on the host with the functions the kernel uses (inspection and tests): first tile of
// every block, totals, and for each probed tile where it lies and which block owns it.
template <int QB>
static int plan_host(const TcParams& p, int grid, long long* first_tile, long long* info, int n_probe, const long long* probe_tiles,
                     long long* probe_out) {
    TileIndex ix;
    int items = 0, longest = 0;
    ix.cum_tiles[0] = 0;
    ix.cum_w[0] = 0;
    for (int b = 0; b < p.B; ++b) {
        int t, w, i, kv;
        plan_sequence<QB>(&ix, p, b, t, w, i, kv);
        ix.cum_tiles[b + 1] = ix.cum_tiles[b] + t;
        ix.cum_w[b + 1] = ix.cum_w[b] + w;
        items += i;
        longest = std::max(longest, kv);
    }
    const int nb = plan_blocks<QB>(&ix, p, grid, items, longest);
    const long long total = (long long)p.H * ix.cum_tiles[p.B], total_w = (long long)p.H * ix.cum_w[p.B];
    for (int c = 0; c <= grid; ++c) first_tile[c] = range_start<QB>(&ix, p, c, nb);
    if (info) { info[0] = total; info[1] = total_w; info[2] = ix.whole_items; info[3] = QB; }
    for (int i = 0; i < n_probe; ++i) {
        long long* o = probe_out + 8 * (size_t)i;
        const long long t = probe_tiles[i];
        if (t < 0 || t >= total) { for (int k = 0; k < 8; ++k) o[k] = -1; continue; }
        Segment sg;
        locate<QB>(&ix, p, t, sg);
        o[0] = sg.b; o[1] = sg.h; o[2] = sg.qb; o[3] = sg.lt; o[4] = sg.Nq; o[5] = sg.Tkv;
        o[6] = ix.whole_items ? -1 : block_of_tile<QB>(&ix, p, t, nb, total_w);
        o[7] = weight_before<QB>(&ix, p, sg);
    }
    return total > 0 ? nb : 0;
}

int tc_plan_host(int B, int H, int G, int N, int L_max, const int32_t* seq_lens, const int32_t* n_active, int grid,
                 long long* first_tile, long long* info, int n_probe, const long long* probe_tiles, long long* probe_out) {
    const int S = tc_stack_for(G, N);
    TcParams p = {};
    p.seq_lens = seq_lens;
    p.n_active = n_active;
    p.B = B; p.H = H / S; p.N = N; p.L_max = L_max;
    p.G = S;
    p.g_shift = S == 8 ? 3 : S == 4 ? 2 : S == 2 ? 1 : 0;
    return chunks_for(N * S) == 10 ? plan_host<kMaxQ>(p, grid, first_tile, info, n_probe, probe_tiles, probe_out)
                                   : plan_host<128>(p, grid, first_tile, info, n_probe, probe_tiles, probe_out);
}

bool tc_supported(const AttentionArgs& a) {
    return tc_shape_supported(a.B, a.H, a.G, a.N, a.D, a.L_max, a.dtype) && encode_fn() != nullptr;
}

size_t tc_workspace_bytes(int, int, int N, int, int) {
    if (N > MCSD_MAX_NODES) return 0;
    return align_up((size_t)2 * kMaxCtas * 2 * kMaxQ * sizeof(float), 256) +
           align_up((size_t)2 * kMaxCtas * kMaxQ * 128 * sizeof(float), 256) + (size_t)65536 * 2 * 4 * sizeof(int);
}

template <int NCH>
static int launch_tc(const TcLaunch& l, cudaStream_t stream) {
    // the opt-in to large dynamic shared memory is per device: done on the first launch on each device
    static std::mutex mu;
    static bool done[64] = {};
    int dev = 0;
    MCSD_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !done[dev]) {
        std::lock_guard<std::mutex> lock(mu);
        MCSD_CUDA_CHECK(cudaFuncSetAttribute(tree_attention_tc_kernel<NCH>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit));
        if (dev >= 0 && dev < 64) done[dev] = true;
    }
    const size_t smem_bytes = 1024 + (size_t)kSlots * kSlotBytes + (size_t)l.p.npadq * 512 + sizeof(TcSmall);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)l.grid);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see the kernel's set-up
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    MCSD_CUDA_CHECK(cudaLaunchKernelEx(&cfg, tree_attention_tc_kernel<NCH>, l.maps[0], l.maps[1], l.maps[2], l.maps[3], l.maps[4],
                                       l.maps[5], l.maps[6], l.maps[7], l.maps[8], l.p));
    return MCSD_OK;
}

int tree_attention_tc(const AttentionArgs& a, WorkspaceHeader* header, void* scratch, size_t scratch_bytes,
                      cudaStream_t stream) {
    if (scratch_bytes < tc_workspace_bytes(a.B, a.H, a.N, a.D, a.L_max)) return MCSD_ERR_WORKSPACE_TOO_SMALL;
    const int S = tc_stack_for(a.G, a.N);       // query heads per work unit
    const int nch = chunks_for(a.N * S);
    const int npadq = nch * 16;
    const int bh = a.B * (a.H / S);             // work units: (sequence, S query heads of one key/value group)
    const int bh_kv = a.B * (a.H / a.G);

    TcLaunch l;
    const bool have_cache = a.L_max > 0;
    bool ok = make_map(&l.maps[0], a.q, a.N, bh, npadq, S);
    ok = ok && make_map(&l.maps[1], have_cache ? a.k_cache : a.k_tree, have_cache ? a.L_max : a.N, bh_kv, kTile);
    ok = ok && make_map(&l.maps[2], have_cache ? a.v_cache : a.v_tree, have_cache ? a.L_max : a.N, bh_kv, kTile);
    ok = ok && make_map(&l.maps[3], a.k_tree, a.N, bh_kv, kTile);
    ok = ok && make_map(&l.maps[4], a.v_tree, a.N, bh_kv, kTile);
    // the same tensors in boxes of 64 rows, for tiles with few rows in use
    ok = ok && make_map(&l.maps[5], have_cache ? a.k_cache : a.k_tree, have_cache ? a.L_max : a.N, bh_kv, kTile / 2);
    ok = ok && make_map(&l.maps[6], have_cache ? a.v_cache : a.v_tree, have_cache ? a.L_max : a.N, bh_kv, kTile / 2);
    ok = ok && make_map(&l.maps[7], a.k_tree, a.N, bh_kv, kTile / 2);
    ok = ok && make_map(&l.maps[8], a.v_tree, a.N, bh_kv, kTile / 2);
    if (!ok) { set_last_cuda_error(cudaErrorInvalidValue); return MCSD_ERR_CUDA; }

    int dev = 0, sms = 0;
    MCSD_CUDA_CHECK(cudaGetDevice(&dev));
    static thread_local int sms_dev = -1, sms_cached = 0;
    if (sms_dev != dev) {
        MCSD_CUDA_CHECK(cudaDeviceGetAttribute(&sms_cached, cudaDevAttrMultiProcessorCount, dev));
        sms_dev = dev;
    }
    sms = sms_cached;
    l.grid = sms < kMaxCtas ? sms : kMaxCtas;

    TcParams& p = l.p;
    p.out = static_cast<__nv_bfloat16*>(a.out);
    p.seq_lens = a.seq_lens;
    p.n_active = a.n_active;
    p.anc = a.anc;
    p.words = a.words;
    p.B = a.B; p.H = a.H / S; p.N = a.N; p.L_max = a.L_max;
    p.G = S;
    p.g_shift = S == 8 ? 3 : S == 4 ? 2 : S == 2 ? 1 : 0;
    p.Hkv = a.H / a.G;
    p.group = a.G;
    p.scale_log2 = a.scale * 1.4426950408889634f;
    p.part_ml = static_cast<float*>(scratch);
    p.part_o = reinterpret_cast<float*>(static_cast<char*>(scratch) + align_up((size_t)2 * kMaxCtas * 2 * kMaxQ * sizeof(float), 256));
    p.counters = reinterpret_cast<int*>(reinterpret_cast<char*>(p.part_o) + align_up((size_t)2 * kMaxCtas * kMaxQ * 128 * sizeof(float), 256));
    p.header = header;
    p.n_slots = kSlots;
    p.npadq = npadq;

    int st;
    switch (nch) {
        case 3: st = launch_tc<3>(l, stream); break;
        case 4: st = launch_tc<4>(l, stream); break;
        case 7: st = launch_tc<7>(l, stream); break;
        case 8: st = launch_tc<8>(l, stream); break;
        default: st = launch_tc<10>(l, stream); break;
    }
    if (st != MCSD_OK) return st;
    count_launches(1);
    return MCSD_OK;
}

}  // namespace mcsd
