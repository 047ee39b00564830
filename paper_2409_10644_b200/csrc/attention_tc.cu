// Tree attention (Section 2.2 of the paper) on the fifth-generation tensor cores of sm_100a: bf16, head_dim 128.
// This file: the kernel for up to 64 query columns per work item (trees of up to 64 nodes per head, or fewer
// nodes with several grouped query heads stacked) and the host side of both tcgen05 kernels; the kernel for wider
// trees is in attention_tc_wide.cu.
//
// One persistent thread block per SM walks a contiguous range of 128-key tiles of the flattened
// (sequence, head, key tile) space, so the K/V stream of every (sequence, head) is read from HBM exactly once
// and all SMs carry the same cost whatever the batch and the prefix lengths are.  Where a range
// boundary cuts a (sequence, head), every side writes an unnormalised partial (running maximum, sum, weighted
// values) and takes a ticket; the block that arrives last combines the partials: split-KV.
//
// The problem is set up transposed so that the small dimension (tree tokens, 16..64 per head) is the MMA N
// and the 128 keys of a tile fill the MMA M:
//     S^T[key][query] = K_tile[key][d] * Q[query][d]^T            (A = K tile, B = Q, both K-major, from TMA)
//     O^T[d][query]  += V_tile[key][d]^T * P^T[key][query]        (A = V tile read MN-major, B = P^T written
//                                                                  by the softmax threads, MN-major)
// Accumulators live in tensor memory: S^T double-buffered (columns 0 and 128), O^T at column 256.
//
// Warp roles (352 threads):
//   warps 0-7  softmax, two warpgroups that split the query columns of each tile: thread r of a group owns
//              key row r of the tile = TMEM lane r.  The running reference maximum of a query is only raised
//              when a score exceeds it by more than 2^8 ("lazy" rescaling): the common tile costs one vote,
//              and only then are exact column maxima reduced (redux.sync inside a warp, shared memory across
//              warps) and O^T in tensor memory rescaled.  Row sums are kept per thread and reduced once per
//              segment.  These threads also apply the tree mask (transposed ancestor bitsets), zero V rows
//              past the end of a ragged tile and run the epilogue.
//   warp 8     TMA producer: K and V tiles into a ring of 32 KB slots, Q once per segment.
//   warp 9     MMA issuer (one thread) and owner of the tensor-memory allocation.
//   warp 10    bookkeeping (one thread): which other blocks share a work item with this one.
// Every mbarrier wait is bounded; a wait that runs out raises a flag in the workspace header, all roles drain
// and the block exits cleanly.
#include <mutex>

#include "attention_tc_common.cuh"

namespace mcsd {

constexpr int kQBlock = 128;                  // queries per work item (this kernel sees at most 64)
constexpr int kSoftmaxGroups = 2;              // warpgroups that split the query columns of every tile
constexpr int kProducerWarp = 4 * kSoftmaxGroups, kMmaWarp = kProducerWarp + 1, kHelperWarp = kMmaWarp + 1;
constexpr int kTcThreads = 32 * (kHelperWarp + 1);
constexpr int kColS1 = 128, kColO = 256;      // tensor-memory columns: S^T twice, O^T
constexpr int kNarrowNodes = 64;              // launches of this kernel have at most 64 stacked queries, so at most 64 nodes

struct TcSmall {
    unsigned long long slot_full[kMaxSlots];
    unsigned long long slot_empty[kMaxSlots];
    unsigned long long s_full[2];
    unsigned long long p_full, pv_done, q_full, q_empty, drain, info_ready;
    uint32_t tmem_base;
    int abort_flag;
    int merge_parts[kSoftmaxGroups];   // > 0: this block finished a split (sequence, head) last and merges it
    // pieces of the (at most two) work items this block shares with others: [0] the segment at the start of its
    // range, [1] the one at the end.  Worked out once by the bookkeeping warp.
    int piece_parts[2];
    unsigned short piece_slot[2][kMaxParts];
    long long range[2];                // first and one-past-last tile of this block
    int n_blocks;                      // blocks that got tiles
    alignas(16) float m_ref[128];
    alignas(16) float alpha[128];      // rescale factors of a slow-path tile; in the epilogue: 1/l (or l) per query
    alignas(16) float wred[kSoftmaxGroups][4][64];
    alignas(16) unsigned long long dmask[kNarrowNodes][3];   // transposed ancestor bitsets: queries that see tree key t
    TileIndex ix;
};
// the small state must leave room for six 32 KB ring slots next to Q and P^T of a 48-query launch
static_assert(sizeof(TcSmall) <= kSmemLimit - 1024 - 6 * 32768 - 48 * 512, "TcSmall grew: the 6-slot ring no longer fits");

// ------------------------------------------------------------------ the kernel
template <int NCH>
__global__ void __launch_bounds__(kTcThreads, 1)
tree_attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kc,
                         const __grid_constant__ CUtensorMap tm_vc, const __grid_constant__ CUtensorMap tm_kt,
                         const __grid_constant__ CUtensorMap tm_vt, const TcParams p) {
    static_assert(NCH <= 4, "wider launches run the kernel of attention_tc_wide.cu");
    constexpr int QB = kQBlock;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int NS = p.n_slots;
    unsigned char* ring = smem;
    unsigned char* p_buf = ring + (size_t)NS * kSlotBytes;
    unsigned char* q_buf = p_buf + (size_t)p.npadq * 256;
    TcSmall* sm = reinterpret_cast<TcSmall*>(q_buf + (size_t)p.npadq * 256);
    const TileIndex* ix = &sm->ix;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;

    // ---- set-up: barriers, tile counts per sequence, this block's range, tensor memory
    if (tid == 0) {
        for (int i = 0; i < kMaxSlots; ++i) { mbar_init(&sm->slot_full[i], 1); mbar_init(&sm->slot_empty[i], 1); }
        mbar_init(&sm->s_full[0], 1);
        mbar_init(&sm->s_full[1], 1);
        mbar_init(&sm->p_full, 128 * kSoftmaxGroups);
        mbar_init(&sm->pv_done, 1);
        mbar_init(&sm->q_full, 1);
        mbar_init(&sm->q_empty, 1);
        mbar_init(&sm->drain, 1);
        mbar_init(&sm->info_ready, 1);
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    plan_ranges<QB>(&sm->ix, p, false, &sm->n_blocks, sm->range);
    const long long total = (long long)p.H * ix->cum_tiles[p.B];
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
        if (lane == 0) {
            long long t = t_begin;
            uint32_t u = 0, seg = 0;
            uint32_t slot = 0, phase = 0;              // ring position of use u (kept incrementally: no divisions)
            bool ok = true;
            while (t < t_end && ok) {
                Segment s;
                locate<QB>(ix, p, t, s);
                const int cnt = (int)min((long long)(s.Tkv - s.lt), t_end - t);
                const int bh = s.b * p.H + s.h;
                const int bh_kv = s.b * p.Hkv + (s.h * p.G) / p.group;
                ok = mbar_wait(&sm->q_empty, (seg & 1u) ^ 1u, abort_flag, hdr, 1);
                if (!ok) break;
                mbar_expect_tx(&sm->q_full, (uint32_t)p.npadq * 256u);
                if (p.G == 1) {
                    tma_load_3d(smem_u32(q_buf), &tm_q, &sm->q_full, 0, s.q0, bh);
                    tma_load_3d(smem_u32(q_buf) + (uint32_t)p.npadq * 128u, &tm_q, &sm->q_full, 64, s.q0, bh);
                } else {
                    // grouped queries: the map is (dim, head of the group, node, sequence x key/value head); a box of
                    // all G heads by npadq / G nodes lands node-major, i.e. as stacked queries q0, q0 + 1, ...
                    tma_load_4d(smem_u32(q_buf), &tm_q, &sm->q_full, 0, 0, s.q0 >> p.g_shift, bh);
                    tma_load_4d(smem_u32(q_buf) + (uint32_t)p.npadq * 128u, &tm_q, &sm->q_full, 64, 0, s.q0 >> p.g_shift, bh);
                }
                for (int i = 0; i < cnt && ok; ++i) {
                    const int lti = s.lt + i;
                    const bool tree = lti >= s.nP;
                    const int row0 = (tree ? lti - s.nP : lti) * kTile;
                    for (int kv = 0; kv < 2 && ok; ++kv, ++u) {
                        ok = mbar_wait(&sm->slot_empty[slot], phase ^ 1u, abort_flag, hdr, 2);
                        if (!ok) break;
                        const CUtensorMap* map = kv == 0 ? (tree ? &tm_kt : &tm_kc) : (tree ? &tm_vt : &tm_vc);
                        const uint32_t dst = smem_u32(ring) + slot * (uint32_t)kSlotBytes;
                        mbar_expect_tx(&sm->slot_full[slot], (uint32_t)kSlotBytes);
                        tma_load_3d(dst, map, &sm->slot_full[slot], 0, row0, bh_kv);
                        tma_load_3d(dst + kSlabBytes, map, &sm->slot_full[slot], 64, row0, bh_kv);
                        if (++slot == (uint32_t)NS) { slot = 0; phase ^= 1u; }
                    }
                }
                t += cnt;
                ++seg;
            }
            if (!ok) {
                // gave up: let copies already issued land before the block exits
                const uint32_t first = u > (uint32_t)NS ? u - (uint32_t)NS : 0u;
                for (uint32_t x = first; x < u; ++x) {
                    void* bar = &sm->slot_full[x % (uint32_t)NS];
                    const uint32_t par = (x / (uint32_t)NS) & 1u;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(bar, par) && clock64() - t0 < kSpinCycles / 8) {}
                }
            }
        }
    } else if (warp == kHelperWarp) {
        // =========================================================== bookkeeping, off everybody's critical path
        if (lane == 0) {
            // which blocks hold the other pieces of the work items this block shares with its neighbours
            for (int which = 0; which < 2; ++which) {
                Segment sp;
                locate<QB>(ix, p, which == 0 ? t_begin : t_end - 1, sp);
                const long long at = which == 0 ? t_begin : t_end - 1;
                const long long t0 = at - sp.lt, t1 = t0 + sp.Tkv;
                int nparts = 0;
                const bool shared = which == 0 ? (t0 < t_begin || t1 > t_end) : (t0 > t_begin && t1 > t_end);
                if (shared) {
                    const int c_lo = block_of_tile<QB>(ix, p, t0, G, total_w, false);
                    const int c_hi = block_of_tile<QB>(ix, p, t1 - 1, G, total_w, false);
                    nparts = min(c_hi - c_lo + 1, kMaxParts);
                    int others = 0;
                    for (int i = 0; i < nparts; ++i) {
                        if (c_lo + i == cta) continue;
                        const long long start = first_tile_of_block<QB>(ix, p, c_lo + i, G, total_w, total, false);
                        sm->piece_slot[which][others++] = (unsigned short)(2 * (c_lo + i) + (t0 > start ? 1 : 0));
                    }
                }
                sm->piece_parts[which] = nparts;
            }
            mbar_arrive(&sm->info_ready);
        }
    } else if (warp == kMmaWarp) {
        // =========================================================== MMA issuer
        if (lane == 0) {
            long long t = t_begin;
            uint32_t g = 0, seg = 0;
            // ring positions of the next K tile (uses 0, 2, 4, ...) and the next V tile (uses 1, 3, 5, ...), kept
            // incrementally: this thread is the pacing one, divisions by the slot count would cost it a tenth
            uint32_t kslot = 0, kphase = 0, vslot = 1u % (uint32_t)NS, vphase = (1u / (uint32_t)NS) & 1u;
            bool ok = true;
            const uint32_t ring_a = smem_u32(ring), q_a = smem_u32(q_buf), p_a = smem_u32(p_buf);
            while (t < t_end && ok) {
                Segment s;
                locate<QB>(ix, p, t, s);
                const int cnt = (int)min((long long)(s.Tkv - s.lt), t_end - t);
                const int npad = (s.Nq + 15) & ~15;
                const uint32_t idesc_s = instr_desc(npad, 0, 0), idesc_pv = instr_desc(npad, 1, 1);
                ok = mbar_wait(&sm->q_full, seg & 1u, abort_flag, hdr, 3);
                for (int i = 0; i <= cnt && ok; ++i) {
                    if (i < cnt) {
                        const uint32_t gi = g + (uint32_t)i, sb = gi & 1u;
                        const uint32_t slot = kslot;
                        ok = mbar_wait(&sm->slot_full[slot], kphase, abort_flag, hdr, 4);
                        if (!ok) break;
                        kslot += 2u;
                        if (kslot >= (uint32_t)NS) { kslot -= (uint32_t)NS; kphase ^= 1u; }
                        tc_fence_after();
                        const uint32_t ka = ring_a + slot * (uint32_t)kSlotBytes;
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            // 16 of the 128 head dims per MMA: slab k/4, 32-byte step inside the swizzled row
                            const uint64_t da = smem_desc(ka + (k >> 2) * kSlabBytes + (k & 3) * 32, 16, 1024, 2);
                            const uint64_t db = smem_desc(q_a + (k >> 2) * (uint32_t)p.npadq * 128u + (k & 3) * 32, 16, 1024, 2);
                            tc_mma(tmem + (sb ? kColS1 : 0), da, db, idesc_s, k > 0);
                        }
                        tc_commit(&sm->s_full[sb]);
                        tc_commit(&sm->slot_empty[slot]);
                        if (i == cnt - 1) tc_commit(&sm->q_empty);
                    }
                    if (i >= 1) {
                        const uint32_t gj = g + (uint32_t)(i - 1);
                        const uint32_t slot = vslot;
                        ok = mbar_wait(&sm->slot_full[slot], vphase, abort_flag, hdr, 5);
                        if (!ok) break;
                        vslot += 2u;
                        if (vslot >= (uint32_t)NS) { vslot -= (uint32_t)NS; vphase ^= 1u; }
                        ok = mbar_wait(&sm->p_full, gj & 1u, abort_flag, hdr, 6);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t va = ring_a + slot * (uint32_t)kSlotBytes;
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            // 16 keys per MMA.  V^T: two 64-dim atoms 16 KB apart (leading), 8-key groups 1 KB apart.
                            const uint64_t da = smem_desc(va + k * 2048, kSlabBytes, 1024, 2);
                            // P^T: 8-key groups 128 B apart (leading), 8-query groups 2 KB apart (stride), no swizzle.
                            const uint64_t db = smem_desc(p_a + k * 256, 128, 2048, 0);
                            tc_mma(tmem + kColO, da, db, idesc_pv, !(i == 1 && k == 0));
                        }
                        tc_commit(&sm->slot_empty[slot]);
                        tc_commit(&sm->pv_done);
                    }
                }
                g += (uint32_t)cnt;
                ++seg;
                t += cnt;
            }
            // all MMAs issued by this thread must have finished before tensor memory is released
            tc_commit(&sm->drain);
            {
                const long long t0 = clock64();
                while (!mbar_try_wait(&sm->drain, 0) && clock64() - t0 < kSpinCycles) {}
            }
        }
    } else {
        // =========================================================== softmax / mask / epilogue
        // Two warpgroups work on the same tile and split its query columns in groups of eight; thread r of
        // either group owns key row r (TMEM lane r).  Per tile the common case is one pass: load S^T, subtract
        // the running reference, check that nothing exceeds it by more than 2^kLazyTau (one vote per group),
        // exponentiate, add to the per-thread row sums and store P^T.  Only when the vote fires (always on the
        // first tile of a segment) are exact column maxima computed and O^T rescaled.
        constexpr int CPT = NCH;                       // 8-column groups per thread (two groups share 16*NCH columns)
        const int wg = warp >> 2, wq = warp & 3;
        const int r = tid & 127;
        const int bar_id = 1 + wg;
        // Reference maxima and rescale factors of this group's own query columns, indexed from the group's first
        // column: the split of the columns between the groups changes with the segment's query count, and one group
        // may already be in the next segment while the other still finishes this one.
        float* const mref = sm->m_ref + 64 * wg;
        float* const alph = sm->alpha + 64 * wg;
        // dmask[t] = set of queries that may see tree key t: the ancestor bitsets transposed.  The bitsets are
        // first copied to shared memory in one coalesced round trip (the P^T buffer is free until the first tile
        // is finished), then the warps transpose them key by key.
        {
            unsigned long long* anc_s = reinterpret_cast<unsigned long long*>(p_buf);
            const int n_words = p.N * p.words;                   // at most 192 * 3 words = 4.5 KB
            for (int i = tid; i < n_words; i += 256) anc_s[i] = p.anc[i];
            asm volatile("bar.sync 3, 256;" ::: "memory");
            // Transposition, one 32-query piece of one key's row per thread and step (consecutive threads take
            // consecutive keys, so a warp reads the same word of 32 bitsets in turn: broadcasts, no bank conflicts).
            // Rows for keys beyond the tree are never read.
            const int NQ = p.N * p.G;                            // stacked queries: query j belongs to node j / G
            const int n_chunks = (NQ + 31) >> 5;
            const uint32_t* anc32 = reinterpret_cast<const uint32_t*>(anc_s);
            for (int idx = tid; idx < p.N * 6; idx += 32 * 4 * kSoftmaxGroups) {
                const int c = idx / p.N, t = idx - c * p.N;
                uint32_t piece = 0;
                if (c < n_chunks) {
                    const uint32_t* col = anc32 + (t >> 5);          // 32-bit half of the 64-bit word that holds bit t
                    const int n_end = min(32, NQ - 32 * c);
#pragma unroll 8
                    for (int i = 0; i < n_end; ++i)
                        piece |= ((col[(size_t)((32 * c + i) >> p.g_shift) * p.words * 2] >> (t & 31)) & 1u) << i;
                }
                reinterpret_cast<uint32_t*>(&sm->dmask[t][0])[c] = piece;
            }
            // both groups read dmask and will overwrite the staging copy: order both before any tile is processed
            asm volatile("bar.sync 3, 256;" ::: "memory");
        }
        const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
        long long t = t_begin;
        uint32_t u = 0, g = 0;
        bool failed = false;
        float acc_l[CPT][8];
        while (t < t_end) {
            Segment s;
            locate<QB>(ix, p, t, s);
            const int cnt = (int)min((long long)(s.Tkv - s.lt), t_end - t);
            const int bh = s.b * p.H + s.h;
            const int ng8 = (s.Nq + 7) >> 3;
            const int half = (ng8 + 1) >> 1;                     // the two groups split the columns evenly
            const int g0 = wg * half;
            const int ncg = wg == 0 ? half : ng8 - half;         // 8-column groups of this thread in this segment
            const int col0 = g0 * 8;
            const unsigned long long nb_lo = s.Nq >= 64 ? ~0ull : ((1ull << s.Nq) - 1ull);
            const unsigned long long nb_hi = s.Nq >= 128 ? ~0ull : (s.Nq > 64 ? ((1ull << (s.Nq - 64)) - 1ull) : 0ull);
            if (r < ncg * 8) mref[r] = -INFINITY;
#pragma unroll
            for (int j = 0; j < CPT; ++j)
#pragma unroll
                for (int k = 0; k < 8; ++k) acc_l[j][k] = 0.f;
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
                    unsigned long long c0 = nb_lo, c1 = nb_hi;
                    if (tree) {                     // bits q0 .. q0+127 of the key's row of the transposed mask
                        c0 &= sm->dmask[row0 + r][s.qb ? 2 : 0];
                        c1 &= s.qb ? 0ull : sm->dmask[row0 + r][1];
                    }
                    cm = col0 >= 64 ? (c1 >> (col0 - 64)) : (col0 == 0 ? c0 : ((c0 >> col0) | (c1 << (64 - col0))));
                }
                if (!mbar_wait(&sm->s_full[sb], (gi >> 1) & 1u, abort_flag, hdr, 7)) failed = true;
                tc_fence_after();
                const uint32_t s_addr = tmem + lane_addr + (sb ? kColS1 : 0) + col0;

                // ---- pass A: scores minus the running reference, and the largest excess
                float y[CPT][8];
                float dmax = -INFINITY;
#pragma unroll
                for (int j = 0; j < CPT; ++j)
                    if (j < ncg) tc_ld8(s_addr + 8 * j, y[j]);
                tc_wait_ld();
#pragma unroll
                for (int j = 0; j < CPT; ++j) {
                    if (j < ncg) {
                        const float4 m0 = *reinterpret_cast<const float4*>(&mref[8 * j]);
                        const float4 m1 = *reinterpret_cast<const float4*>(&mref[8 * j + 4]);
                        const float mr[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
                        const uint32_t bits = (uint32_t)(cm >> (8 * j)) & 0xFFu;
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            float yy = fmaf(y[j][k], p.scale_log2, -mr[k]);
                            if (!full_tile && !((bits >> k) & 1u)) yy = -INFINITY;
                            dmax = fmaxf(dmax, yy);
                            y[j][k] = yy;
                        }
                    }
                }
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
                    if (gi > 0 && !mbar_wait(&sm->pv_done, (gi - 1u) & 1u, abort_flag, hdr, 8)) failed = true;
                    if (rescale) {
                        tc_fence_after();
#pragma unroll
                        for (int j = 0; j < CPT; ++j) {
                            if (j < ncg) {
                                float o[8];
                                tc_ld8(tmem + lane_addr + kColO + col0 + 8 * j, o);
                                tc_wait_ld();
#pragma unroll
                                for (int k = 0; k < 8; ++k) {
                                    const float a = alph[8 * j + k];
                                    o[k] *= a;
                                    acc_l[j][k] *= a;
                                }
                                tc_st8(tmem + lane_addr + kColO + col0 + 8 * j, o);
                            }
                        }
                        tc_wait_st();
                    }
#pragma unroll
                    for (int j = 0; j < CPT; ++j) {
                        if (j < ncg) {
                            float v[8];
                            tc_ld8(s_addr + 8 * j, v);
                            tc_wait_ld();
                            const uint32_t bits = (uint32_t)(cm >> (8 * j)) & 0xFFu;
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                float yy = fmaf(v[k], p.scale_log2, -mref[8 * j + k]);
                                if (!full_tile && !((bits >> k) & 1u)) yy = -INFINITY;
                                y[j][k] = yy;
                            }
                        }
                    }
                }

                // P buffer must no longer be read by the previous tile's MMA; this wait also keeps every thread
                // within one phase of the p_full barrier
                if (gi > 0 && !mbar_wait(&sm->pv_done, (gi - 1u) & 1u, abort_flag, hdr, 8)) failed = true;

                // ---- pass B: probabilities, row sums, P^T for the second MMA
#pragma unroll
                for (int j = 0; j < CPT; ++j) {
                    if (j < ncg) {
                        uint32_t packed[4];
#pragma unroll
                        for (int k = 0; k < 8; k += 2) {
                            // 2^-inf = 0 for masked entries
                            const float p0 = ex2_approx(y[j][k]), p1 = ex2_approx(y[j][k + 1]);
                            acc_l[j][k] += p0;
                            acc_l[j][k + 1] += p1;
                            __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
                            packed[k >> 1] = *reinterpret_cast<uint32_t*>(&h2);
                        }
                        *reinterpret_cast<uint4*>(p_buf + (size_t)(g0 + j) * 2048 + (size_t)r * 16) =
                            make_uint4(packed[0], packed[1], packed[2], packed[3]);
                    }
                }
                // rows of the V tile past the end of the prefix / tree may hold anything: make them zero
                if (wg == 0 && valid < kTile) {
                    const uint32_t uv = u + 2u * (uint32_t)i + 1u, slot = uv % (uint32_t)NS;
                    if (!mbar_wait(&sm->slot_full[slot], (uv / (uint32_t)NS) & 1u, abort_flag, hdr, 9)) failed = true;
                    if (r >= valid && !failed) {
                        uint4* z0 = reinterpret_cast<uint4*>(ring + (size_t)slot * kSlotBytes + (size_t)r * 128);
                        uint4* z1 = reinterpret_cast<uint4*>(ring + (size_t)slot * kSlotBytes + kSlabBytes + (size_t)r * 128);
#pragma unroll
                        for (int x = 0; x < 8; ++x) { z0[x] = make_uint4(0, 0, 0, 0); z1[x] = make_uint4(0, 0, 0, 0); }
                    }
                }
                fence_async_smem();
                tc_fence_before();
                mbar_arrive(&sm->p_full);
            }
            if (group_sync_any(bar_id, failed)) { failed = true; break; }

            // ---- epilogue of the segment: each group finishes its own query columns
            const uint32_t glast = g + (uint32_t)cnt - 1u;
            const bool full = (cnt == s.Tkv);
            const int slot_id = 2 * cta + (t > t_begin ? 1 : 0);
            if (!mbar_wait(&sm->pv_done, glast & 1u, abort_flag, hdr, 10)) failed = true;
            tc_fence_after();
            // Row sums: every thread holds a partial sum per query; reduce the 8 sums of a column group across the
            // warp by recursive halving (9 shuffles instead of 40): after the three exchange steps lane L holds the
            // sum of column (L >> 2) & 7 over its exchange partners, two more steps finish the reduction.
#pragma unroll
            for (int j = 0; j < CPT; ++j) {
                if (j < ncg) {
                    float v4[4], v2[2], v1;
                    {
                        const bool up = lane & 16;
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const float send = up ? acc_l[j][k] : acc_l[j][k + 4];
                            const float keep = up ? acc_l[j][k + 4] : acc_l[j][k];
                            v4[k] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
                        }
                    }
                    {
                        const bool up = lane & 8;
#pragma unroll
                        for (int k = 0; k < 2; ++k) {
                            const float send = up ? v4[k] : v4[k + 2];
                            const float keep = up ? v4[k + 2] : v4[k];
                            v2[k] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
                        }
                    }
                    {
                        const bool up = lane & 4;
                        const float send = up ? v2[0] : v2[1];
                        const float keep = up ? v2[1] : v2[0];
                        v1 = keep + __shfl_xor_sync(0xffffffffu, send, 4);
                    }
                    v1 += __shfl_xor_sync(0xffffffffu, v1, 2);
                    v1 += __shfl_xor_sync(0xffffffffu, v1, 1);
                    // lane bits 4,3,2 select column 4*b4 + 2*b3 + b2
                    if ((lane & 3) == 0) sm->wred[wg][wq][8 * j + ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1)] = v1;
                }
            }
            if (group_sync_any(bar_id, failed)) { failed = true; break; }
            if (r < ncg * 8) {
                const float l = (sm->wred[wg][0][r] + sm->wred[wg][1][r]) + (sm->wred[wg][2][r] + sm->wred[wg][3][r]);
                if (full) {
                    alph[r] = l > 0.f ? 1.f / l : 0.f;
                } else {
                    alph[r] = l;                   // kept for the merge below
                    p.part_ml[((size_t)slot_id * 2 + 0) * kMaxQ + col0 + r] = mref[r];
                    p.part_ml[((size_t)slot_id * 2 + 1) * kMaxQ + col0 + r] = l;
                }
            }
            group_sync_any(bar_id, false);
            // O^T rows of this thread, up to four column groups per tensor-memory round trip
            constexpr int EB = CPT < 4 ? CPT : 4;
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
                        if (j0 + jj < CPT && j0 + jj < ncg) {
                            if (full) {
                                // Thread r holds head dim r of eight queries.  An 8 x 8 transpose inside every group
                                // of eight lanes (three butterfly stages) leaves lane 8a + k with eight consecutive
                                // head dims of query k: one 16-byte store per thread instead of eight 2-byte ones.
                                // (The same for the fp32 partials measured no faster.)
                                float v[8];
#pragma unroll
                                for (int k = 0; k < 8; ++k) v[k] = o[jj][k] * alph[8 * (j0 + jj) + k];
#pragma unroll
                                for (int m = 4; m > 0; m >>= 1) {
                                    const bool up = lane & m;
#pragma unroll
                                    for (int i = 0; i < 8; ++i) {
                                        if (i & m) continue;
                                        const float send = up ? v[i] : v[i | m];
                                        const float got = __shfl_xor_sync(0xffffffffu, send, m);
                                        if (up) v[i] = got; else v[i | m] = got;
                                    }
                                }
                                const int n = col0 + 8 * (j0 + jj) + (lane & 7);
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
                                    const int n = col0 + 8 * (j0 + jj) + k;
                                    if (n < s.Nq) p.part_o[((size_t)slot_id * kMaxQ + n) * 128 + r] = o[jj][k];
                                }
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            if (!full) {
                // Split-KV combine: every block that finished a piece of this work item takes a ticket; the last
                // one merges the other pieces (read back from the workspace) with its own, which is still in
                // tensor memory.  The two softmax groups own disjoint query columns and run this protocol independently.
                __threadfence();
                group_sync_any(bar_id, false);
                const int which = slot_id & 1;
                if (r == 0) {
                    if (!mbar_wait(&sm->info_ready, 0, abort_flag, hdr, 12)) failed = true;
                    int* counter = p.counters + ((size_t)bh * 2 + s.qb) * 4 + wg;
                    const int nparts = sm->piece_parts[which];
                    sm->merge_parts[wg] = nparts;
                    const int old = atomicAdd(counter, 1);
                    if (old == nparts - 1) {
                        *(volatile int*)counter = 0;              // nobody else arrives in this launch: ready for the next one
                        __threadfence();                          // acquire: the other pieces' partials are visible
                    } else {
                        sm->merge_parts[wg] = 0;                  // not the last: nothing more to do
                    }
                }
                group_sync_any(bar_id, false);
                const int nparts = sm->merge_parts[wg];
                if (nparts > 0) {
                    // The other pieces sit in the workspace behind a memory system that is busy streaming keys and
                    // values, so what counts is the number of dependent round trips: one per piece and batch of
                    // column groups.  All O^T loads of a piece are issued first; while they are in flight the thread
                    // that owns a query column fetches the piece's (m, l) for it, folds them into its running
                    // reference and normaliser and leaves the two rescale factors of that column in shared memory;
                    // after a group barrier every thread applies them to its rows.
                    const int np1 = nparts - 1;
                    float* const fa = &sm->wred[wg][0][0];                   // [piece parity][64]: factor for what we have
                    float* const fw = &sm->wred[wg][2][0];                   // [piece parity][64]: factor for the new piece
                    const bool col_owner = r < ncg * 8 && col0 + r < s.Nq;
                    constexpr int GB = CPT < 4 ? CPT : 2;                    // column groups per batch (what the registers allow)
#pragma unroll
                    for (int j0 = 0; j0 < CPT; j0 += GB) {
                        if (j0 >= ncg) break;
                        float acc[GB][8];
#pragma unroll
                        for (int jj = 0; jj < GB; ++jj)
                            if (j0 + jj < CPT && j0 + jj < ncg) tc_ld8(tmem + lane_addr + kColO + col0 + 8 * (j0 + jj), acc[jj]);
                        tc_wait_ld();
                        float m_run = col_owner ? mref[r] : -INFINITY;       // of column r, kept by its owner
                        float l_run2 = col_owner ? alph[r] : 0.f;
                        for (int i = 0; i < np1; ++i) {
                            const int slot = sm->piece_slot[which][i];
                            float os[GB][8];
#pragma unroll
                            for (int jj = 0; jj < GB; ++jj)
#pragma unroll
                                for (int k = 0; k < 8; ++k) {
                                    const int n = col0 + 8 * (j0 + jj) + k;
                                    const bool on = j0 + jj < CPT && j0 + jj < ncg && n < s.Nq;
                                    os[jj][k] = on ? __ldcg(p.part_o + ((size_t)slot * kMaxQ + n) * 128 + r) : 0.f;
                                }
                            float* const fa_i = fa + 64 * (i & 1);
                            float* const fw_i = fw + 64 * (i & 1);
                            if (col_owner) {
                                const float ms = __ldcg(p.part_ml + ((size_t)slot * 2 + 0) * kMaxQ + col0 + r);
                                const float ls = __ldcg(p.part_ml + ((size_t)slot * 2 + 1) * kMaxQ + col0 + r);
                                const float mn = fmaxf(m_run, ms);
                                const float a = (mn == -INFINITY || m_run == -INFINITY) ? 0.f : exp2f(m_run - mn);
                                const float wgt = (mn == -INFINITY || ms == -INFINITY) ? 0.f : exp2f(ms - mn);
                                l_run2 = l_run2 * a + ls * wgt;
                                m_run = mn;
                                fa_i[r] = a;
                                fw_i[r] = wgt;
                            }
                            group_sync_any(bar_id, false);                   // factors of piece i are in place
#pragma unroll
                            for (int jj = 0; jj < GB; ++jj)
#pragma unroll
                                for (int k = 0; k < 8; ++k) {
                                    const int rel = 8 * (j0 + jj) + k;
                                    if (j0 + jj < CPT && j0 + jj < ncg)
                                        acc[jj][k] = fmaf(os[jj][k], fw_i[rel], acc[jj][k] * fa_i[rel]);
                                }
                            // piece i + 2 reuses these factor slots: by then every thread has passed the barrier of
                            // piece i + 1, which it reaches only after the loop above
                        }
                        // normaliser of every column, then the output rows
                        group_sync_any(bar_id, false);                       // everybody is done with the factor slots
                        if (col_owner) fa[r] = l_run2 > 0.f ? 1.f / l_run2 : 0.f;
                        group_sync_any(bar_id, false);
#pragma unroll
                        for (int jj = 0; jj < GB; ++jj)
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                const int rel = 8 * (j0 + jj) + k, n = col0 + rel;
                                if (j0 + jj < CPT && j0 + jj < ncg && n < s.Nq) {
                                    const int jq = s.q0 + n;
                                    p.out[(((size_t)bh * p.G + (jq & (p.G - 1))) * p.N + (jq >> p.g_shift)) * 128 + r] =
                                        __float2bfloat16_rn(acc[jj][k] * fa[rel]);
                                }
                            }
                        group_sync_any(bar_id, false);                       // before the next batch reuses the slots
                    }
                }
            }
            group_sync_any(bar_id, false);
            g += (uint32_t)cnt;
            u += 2u * (uint32_t)cnt;
            t += cnt;
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

// Padded query columns of a launch in 16-column chunks: 3 or 4 for the kernel above, 7, 8 or 10 for the wide one
// (10 = 160 queries in one pass; trees with more stacked queries are cut into blocks of 160).
static int chunks_for(int nq) {
    const int nch = ((nq < kMaxQ ? nq : kMaxQ) + 15) / 16;
    return nch <= 3 ? 3 : nch <= 4 ? 4 : nch <= 7 ? 7 : nch <= 8 ? 8 : 10;
}

static int slots_for(int nch) {
    const long long avail = (long long)kSmemLimit - 1024 - (long long)sizeof(TcSmall) - (long long)nch * 16 * 512;
    long long ns = avail / kSlotBytes;
    if (ns > kMaxSlots) ns = kMaxSlots;
    return (int)ns;
}

// Query heads of one key/value group stacked into one work unit: the largest of 8, 4, 2, 1 that divides the group
// and keeps the stacked queries within one query block (a second block would stream the keys again, which is what
// a second unit does as well, with narrower tiles).
static int tc_stack_for(int G, int N) {
    for (int s = 8; s > 1; s >>= 1)
        if (G % s == 0 && s * N <= kMaxQ) return s;
    return 1;
}

// The per-sequence prefix sums of tiles and cost units are 32-bit: bound the largest launch so that they cannot
// wrap (a sequence of L_max keys and 192 nodes costs at most 2 * (tiles + 4) * 64 units per head).
bool tc_supported(const AttentionArgs& a) {
    if (!(a.G >= 1 && a.H % a.G == 0 && a.N <= MCSD_MAX_NODES && a.B <= kMaxBatchTc && encode_fn() != nullptr)) return false;
    const long long tiles = (long long)a.L_max / kTile + 4;
    return (long long)a.B * tiles * 2 * 64 < (1LL << 30);
}

size_t tc_workspace_bytes(int, int, int N, int, int) {
    if (N > MCSD_MAX_NODES) return 0;
    return align_up((size_t)2 * kMaxCtas * 2 * kMaxQ * sizeof(float), 256) +
           align_up((size_t)2 * kMaxCtas * kMaxQ * 128 * sizeof(float), 256) + (size_t)65536 * 2 * 4 * sizeof(int);
}

template <int NCH>
static int launch_tc(const TcLaunch& l, size_t smem_bytes, cudaStream_t stream) {
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
    tree_attention_tc_kernel<NCH><<<l.grid, kTcThreads, smem_bytes, stream>>>(l.maps[0], l.maps[1], l.maps[2], l.maps[3], l.maps[4], l.p);
    MCSD_CUDA_CHECK(cudaGetLastError());
    return MCSD_OK;
}

int tree_attention_tc(const AttentionArgs& a, WorkspaceHeader* header, void* scratch, size_t scratch_bytes,
                      cudaStream_t stream) {
    if (scratch_bytes < tc_workspace_bytes(a.B, a.H, a.N, a.D, a.L_max)) return MCSD_ERR_WORKSPACE_TOO_SMALL;
    const int S = tc_stack_for(a.G, a.N);       // query heads per work unit
    const int nch = chunks_for(a.N * S);
    const int npadq = nch * 16;
    const bool wide = nch > 4;
    const int ns = wide ? slots_for_wide(nch) : slots_for(nch);
    if (ns < 4) return MCSD_ERR_BAD_SHAPE;
    const int bh = a.B * (a.H / S);             // work units: (sequence, S query heads of one key/value group)
    const int bh_kv = a.B * (a.H / a.G);

    TcLaunch l;
    const bool have_cache = a.L_max > 0;
    bool ok = make_map(&l.maps[0], a.q, a.N, bh, npadq, S);
    ok = ok && make_map(&l.maps[1], have_cache ? a.k_cache : a.k_tree, have_cache ? a.L_max : a.N, bh_kv, kTile);
    ok = ok && make_map(&l.maps[2], have_cache ? a.v_cache : a.v_tree, have_cache ? a.L_max : a.N, bh_kv, kTile);
    ok = ok && make_map(&l.maps[3], a.k_tree, a.N, bh_kv, kTile);
    ok = ok && make_map(&l.maps[4], a.v_tree, a.N, bh_kv, kTile);
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
    p.n_slots = ns;
    p.npadq = npadq;

    int st;
    if (wide) {
        st = launch_tc_wide(nch, l, stream);
    } else {
        const size_t smem_bytes = 1024 + (size_t)ns * kSlotBytes + (size_t)npadq * 512 + sizeof(TcSmall);
        st = nch == 3 ? launch_tc<3>(l, smem_bytes, stream) : launch_tc<4>(l, smem_bytes, stream);
    }
    if (st != MCSD_OK) return st;
    count_launches(1);
    return MCSD_OK;
}

}  // namespace mcsd
