/*
 * mcsd.h -- C ABI of libmcsd: one-pass verification of a candidate token tree
 * (multi-candidate speculative decoding) on one NVIDIA B200 (sm_100a).
 *
 * Three operations make up the verification step of the generation loop in Fig. 1 of
 * "Improving Multi-candidate Speculative Decoding" (steps 2, 4, 5 and the sampling of step 6):
 *
 *   mcsd_build_mask      topology-aware causal mask of the token tree, built once (Sections 2.2, 3.2)
 *   mcsd_tree_attention  attention of all tree tokens over the prefix KV cache plus the tree's own
 *                        keys/values under that mask (tree attention, Section 2.2)
 *   mcsd_verify_tree     multi-candidate accept/reject walk, longest-sequence selection and sampling of
 *                        the new token (Fig. 1 steps 4-6; Section 3.1 for several target-initialised roots)
 *
 * Conventions
 *   - Every function returns an int status: MCSD_OK (0) or a negative MCSD_ERR_* code.  Nothing throws or
 *     aborts.  mcsd_status_string() names a code; mcsd_last_cuda_error() returns the cudaError_t behind the
 *     most recent MCSD_ERR_CUDA of the calling thread.
 *   - Pointers marked [dev] are device pointers owned by the caller; pointers marked [host] are host
 *     pointers.  All tensors are dense and contiguous in the stated layout.  These functions never allocate
 *     or free device memory: kernels that need scratch take a caller-supplied workspace whose size the
 *     matching *_workspace_bytes() query returns.  A workspace is 256-byte aligned and must be zero-filled
 *     once before its first use (its first 256 bytes hold a sticky status word, see mcsd_workspace_status).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls only enqueue
 *     work on that stream and never synchronise, except where stated.
 *   - Nodes of the tree are in level (BFS) order: parent[n] < n, depth non-decreasing in n, children of a
 *     node contiguous.  Roots carry parent -1 and form level 0.  With one root the tree is
 *     draft-initialised and node 0 is the last emitted token; with R > 1 roots it is the
 *     target-initialised forest of Section 3.1 whose roots are accepted by construction.
 *   - The dynamic sliced mask of Section 3.2 is a row count: keeping the first gamma draft levels keeps the
 *     first n_active = level_start[gamma + 1] nodes, and in level order no kept row has a bit beyond them.
 */
#ifndef MCSD_H_
#define MCSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MCSD_OK                        0
#define MCSD_ERR_NULL                 -1  /* a required pointer is NULL */
#define MCSD_ERR_BAD_SHAPE            -2  /* a size or an alignment is out of the supported range */
#define MCSD_ERR_NOT_BFS              -3  /* parent array is not a level-ordered forest */
#define MCSD_ERR_BAD_DTYPE            -4
#define MCSD_ERR_WORKSPACE_TOO_SMALL  -5
#define MCSD_ERR_CUDA                 -6  /* a CUDA runtime/driver call failed; see mcsd_last_cuda_error() */
#define MCSD_ERR_TIMEOUT              -7  /* a bounded device-side wait ran out (reported by mcsd_workspace_status) */
#define MCSD_ERR_STATIC_LIMIT         -8  /* problem exceeds the built-in scratch of a *_static entry point */

#define MCSD_MAX_NODES   192              /* largest tree (roots included) */
#define MCSD_MAX_WORDS   3                /* 64-bit mask words per node for MCSD_MAX_NODES */

#define MCSD_BF16  0
#define MCSD_F32   1

const char* mcsd_status_string(int status);
int mcsd_last_cuda_error(void);

/*
 * Number of kernels this process has launched through the library so far (all threads, all devices).
 * Bookkeeping for benchmarks that report how many launches a step of Fig. 1's verification costs.
 */
long long mcsd_launch_count(void);

/*
 * Topology-aware causal mask (Section 2.2; Fig. 1 step 2), built once for the deepest tree (Section 3.2).
 *
 *   parent_host      [host] int32[n_nodes], level order, -1 for roots.  Validated on the CPU before anything
 *                    is launched; a bad array returns MCSD_ERR_NOT_BFS and touches no output.
 *   anc_dev          [dev]  uint64[n_nodes][words]: bit (j % 64) of word (j / 64) of row n is set iff tree
 *                    token n may attend to tree token j, i.e. j is n or an ancestor of n.
 *   words            must be >= ceil(n_nodes / 64) and <= MCSD_MAX_WORDS; unused high words are zeroed.
 *   depth_dev        [dev]  int32[n_nodes], level of every node (roots 0): position = prefix length + depth.
 *   level_start_dev  [dev]  int32[n_nodes + 1] capacity; entries 0..*n_levels are written:
 *                    level_start[l] = index of the first node of level l, level_start[n_levels] = n_nodes.
 *                    May be NULL.
 *   level_start_host [host] same content, capacity n_nodes + 1.  May be NULL.
 *   n_levels         [host] out, number of levels.  May be NULL.
 *
 * The tree travels to the kernel as a launch argument, so no host-to-device copy and no synchronisation
 * takes place; outputs are ready when the work enqueued on `stream` completes.
 * Errors: MCSD_ERR_NULL, MCSD_ERR_BAD_SHAPE (n_nodes < 1 or > MCSD_MAX_NODES, bad words), MCSD_ERR_NOT_BFS,
 * MCSD_ERR_CUDA.
 */
int mcsd_build_mask(const int32_t* parent_host, int n_nodes,
                    uint64_t* anc_dev, int words,
                    int32_t* depth_dev,
                    int32_t* level_start_dev, int32_t* level_start_host, int* n_levels,
                    void* stream);

/*
 * Tree attention (Section 2.2): for every sequence b, head h and active tree token n < n_active[b]
 *     out[b][h][n] = sum_j softmax_j(softmax_scale * <q[b][h][n], k_j>) v_j
 * over the prefix keys j = 0 .. seq_lens[b]-1 of the cache and the tree keys j with bit j set in anc[n].
 * Rows n >= n_active[b] of `out` are not written.
 *
 *   q, k_tree, v_tree, out  [dev] [B][H][N][D]
 *   k_cache, v_cache        [dev] [B][H][L_max][D]; only the first seq_lens[b] rows of sequence b are used
 *                           (later rows may hold anything, NaN bit patterns included)
 *   seq_lens                [dev] int32[B], 0 <= seq_lens[b] <= L_max
 *   n_active                [dev] int32[B], 0 <= n_active[b] <= N (a level-order prefix of the tree), or NULL = N;
 *                           rows n >= n_active[b] of k_tree and v_tree are not used and may hold anything
 *   anc, words              the mask from mcsd_build_mask for the N-node tree
 *   D                       64 or 128;  N <= MCSD_MAX_NODES;  B * H <= 65535
 *   dtype                   MCSD_BF16: bf16 storage, fp32 softmax and accumulation (tensor-core products when
 *                           D == 128, all tensors are 16-byte aligned and the shape is one that
 *                           mcsd_tree_attention_path() reports as MCSD_PATH_TENSOR_CORE);  MCSD_F32: fp32 throughout
 *   workspace               [dev] scratch of at least mcsd_tree_attention_workspace_bytes(...) bytes; holds
 *                           split-KV partial results and the status word.  Calls that may overlap on the
 *                           device need distinct workspaces.
 *
 * Split-KV: the keys of one (b, h) may be processed by several thread blocks, each producing an
 * unnormalised partial (running maximum, sum, weighted values); a combine pass merges them.
 * Errors: MCSD_ERR_NULL, MCSD_ERR_BAD_SHAPE, MCSD_ERR_BAD_DTYPE, MCSD_ERR_WORKSPACE_TOO_SMALL, MCSD_ERR_CUDA.
 * Device-side waits are bounded; one that runs out is reported later by mcsd_workspace_status().
 */
size_t mcsd_tree_attention_workspace_bytes(int B, int H, int N, int D, int L_max, int dtype);

int mcsd_tree_attention(const void* q, const void* k_cache, const void* v_cache,
                        const void* k_tree, const void* v_tree, void* out,
                        const int32_t* seq_lens, const int32_t* n_active,
                        const uint64_t* anc, int words,
                        int B, int H, int N, int D, int L_max, float softmax_scale,
                        int dtype, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Self-test of the bounded device-side waits (the paper has no counterpart; the kernels of mcsd_tree_attention wait on
 * hardware barriers for tiles, products and partial results, and every such wait has a limit so that a lost signal ends
 * in a status, not in a hung GPU).  Launches one small block that waits, with the same wait routine, for a signal that
 * never comes: after about `microseconds` (1 .. 100000) the wait gives up, the block exits normally, and the workspace
 * header holds MCSD_ERR_TIMEOUT, which mcsd_workspace_status() then returns.  The workspace must be zero-filled again
 * before it is used for anything else.  Nothing faults, traps or spins without limit.
 *   workspace   [dev] >= 256 bytes, 256-byte aligned
 * Errors: MCSD_ERR_NULL, MCSD_ERR_BAD_SHAPE, MCSD_ERR_CUDA.
 */
int mcsd_selftest_bounded_wait(void* workspace, size_t workspace_bytes, int microseconds, void* stream);

/*
 * Which kernel mcsd_tree_attention / mcsd_tree_attention_gqa runs for a shape (Section 2.2 defines the operation; the
 * choice of kernel is this library's).  The tensor-core kernel (tcgen05, bandwidth-bound) takes bf16, D = 128,
 * B <= 256 and B * (L_max / 128 + 4) < 2^23 (its per-sequence tables are 32-bit and live in shared memory); every
 * other valid shape -- fp32, D = 64, larger batches, longer prefixes -- runs the CUDA-core kernel, which is
 * arithmetic-bound and several times slower per key.  A caller with more than 256 sequences gets the fast kernel by
 * splitting the batch over several calls.  Host only, no CUDA call.
 *
 * Returns MCSD_PATH_TENSOR_CORE or MCSD_PATH_CUDA_CORE, or a negative status (MCSD_ERR_BAD_SHAPE, MCSD_ERR_BAD_DTYPE)
 * for a shape mcsd_tree_attention rejects.  (Tensors that are not 16-byte aligned also take the CUDA-core kernel.)
 */
#define MCSD_PATH_CUDA_CORE 0
#define MCSD_PATH_TENSOR_CORE 1
int mcsd_tree_attention_path(int B, int H_q, int H_kv, int N, int D, int L_max, int dtype);

/*
 * How the tensor-core kernel would cut a launch among its thread blocks (the paper has no counterpart: Section 2.2
 * defines the attention, the schedule is this library's).  The key/value tiles of a launch are numbered in the
 * order (sequence, work unit, query block, 128-key tile; prefix tiles before tree tiles); thread block c processes
 * tiles first_tile[c] .. first_tile[c + 1] - 1, ranges of about equal estimated cost, or whole work items when the
 * launch is small.  The kernel evaluates the same functions on the device; this entry point evaluates them on the
 * host, for inspection and tests.  Host only, no CUDA call; all pointers are host pointers.
 *
 *   seq_lens, n_active   [host] int32[B] as for mcsd_tree_attention (n_active may be NULL = N)
 *   n_blocks             thread blocks of the launch, 1 .. 160 (the kernel uses one per multiprocessor)
 *   first_tile           [host] int64[n_blocks + 1], written; blocks past the returned count get empty ranges
 *   info                 [host] int64[4] or NULL, written: tiles in the launch, their total cost in the kernel's
 *                        units, 1 if blocks take whole work items, queries per work item at most (128 or 160)
 *   probe_tiles          [host] int64[n_probe] tile numbers to describe (n_probe may be 0)
 *   probe_out            [host] int64[n_probe][8], written: sequence, work unit within the sequence, query block, tile
 *                        within the work item, queries of the work item, tiles of the work item, owning block as the
 *                        merging block computes it (-1 in whole-item mode), cost of the tiles before it;
 *                        eight times -1 for a tile number outside the launch
 *
 * Returns the number of blocks that get work (0 for a launch without keys), MCSD_ERR_BAD_SHAPE for a shape the
 * tensor-core kernel does not take (see mcsd_tree_attention_path) or a bad n_blocks, MCSD_ERR_NULL, or the status
 * mcsd_tree_attention_path returns for an invalid shape.
 */
int mcsd_tree_attention_plan(int B, int H_q, int H_kv, int N, int D, int L_max, int dtype, const int32_t* seq_lens,
                             const int32_t* n_active, int n_blocks, int64_t* first_tile, int64_t* info, int n_probe,
                             const int64_t* probe_tiles, int64_t* probe_out);

/*
 * mcsd_tree_attention for a target with grouped-query attention: q and out have H_q heads, the four key/value
 * tensors H_kv heads, H_q = G * H_kv, and query head h reads key/value head h / G (the paper's targets are
 * multi-head models, G = 1; Section 2.2 defines the attention itself).  Everything else as mcsd_tree_attention.
 * With bf16 and head_dim 128 the tensor-core kernel stacks the queries of S heads of a group into one work unit
 * (S the largest of 8, 4, 2 that divides G with S * N <= 160, the most query columns one pass over the keys takes;
 * else 1), so that a key/value head is streamed G / S times instead of G times.
 *
 *   q, out                  [dev] dtype[B][H_q][N][D]
 *   k_cache, v_cache        [dev] dtype[B][H_kv][L_max][D]
 *   k_tree, v_tree          [dev] dtype[B][H_kv][N][D]
 *   workspace               >= mcsd_tree_attention_workspace_bytes(B, H_q, N, D, L_max, dtype) bytes, zero-filled once
 *
 * Errors: as mcsd_tree_attention, plus MCSD_ERR_BAD_SHAPE when H_q is not a multiple of H_kv.
 */
int mcsd_tree_attention_gqa(const void* q, const void* k_cache, const void* v_cache,
                            const void* k_tree, const void* v_tree, void* out,
                            const int32_t* seq_lens, const int32_t* n_active,
                            const uint64_t* anc, int words,
                            int B, int H_q, int H_kv, int N, int D, int L_max,
                            float softmax_scale, int dtype,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * Reads the status word that kernels of mcsd_tree_attention / mcsd_verify_tree leave in `workspace`.
 * The word is sticky: kernels only ever set it, the caller clears it by zero-filling the first 256 bytes.
 * Synchronises `stream`.  Returns MCSD_OK, MCSD_ERR_TIMEOUT (a bounded wait ran out; outputs of that call
 * are invalid) or MCSD_ERR_CUDA.
 */
int mcsd_workspace_status(const void* workspace, void* stream);

/*
 * Multi-candidate accept/reject (Fig. 1 steps 4-6).  For every sequence and every root the walk starts at
 * the root; at node u the children c_1..c_k are tried in order: child c_i with token x_i is accepted iff
 *     u_accept[c_i] < min(1, pt(x_i) / q_u(x_i))
 * where pt starts as p_u and after every rejection becomes norm(max(pt - q_u, 0)).  The first accepted child
 * becomes the new u (with pt reset to its own row); if none is accepted, or u has no children within the
 * first gamma[b] draft levels, the walk stops at u and one more token is drawn from the distribution it
 * stopped with (pt, or p_u at a leaf) by inverse CDF in token-id order: the smallest t with
 * cumsum(dist)[t] > u_bonus[u] * sum(dist).  The root with the longest accepted path wins (ties: lowest index).
 *
 *   p, q          [dev] float[B][N][V]: row n is the target / draft next-token distribution after node n
 *   tokens        [dev] int32[B][N]: token id of every node (root tokens are never tested)
 *   parent        [dev] int32[N]: the array given to mcsd_build_mask
 *   level_start   [dev] int32[n_levels + 1] from mcsd_build_mask
 *   n_roots       number of level-0 nodes
 *   gamma         [dev] int32[B], draft levels kept per sequence (0..n_levels-1), or NULL = all
 *   u_accept      [dev] float[B][N] uniforms, one per candidate node
 *   u_bonus       [dev] float[B][N] uniforms, one per possible stop node
 *   accept_len    [dev] int32[B] out: accepted draft tokens of the winning path
 *   out_tokens    [dev] int32[B][n_levels + 1] out: (token of the winning root if n_roots > 1,) accepted
 *                 tokens, new token; padded with -1
 *   out_nodes     [dev] int32[B][n_levels] out: accepted node ids, padded with -1
 *   best_root     [dev] int32[B] out
 *   next_roots    [dev] int32[B][R] out or NULL: the R most probable ids of the distribution the new token
 *                 was drawn from (ties to the smaller id) -- the candidates with which a target-initialised
 *                 tree (Section 3.1) seeds its next step
 *   workspace     [dev] >= mcsd_verify_tree_workspace_bytes(B, N, V) bytes, zero-filled before its first use (it
 *                 holds a per-sequence arrival counter that every call leaves at zero again)
 *
 * One launch on `stream`: one block per (sequence, node) decides the accepted child of every node; the block
 * that finishes a sequence's last node (an arrival counter per sequence, nothing waits) follows the paths and
 * draws the new token.
 *
 * Errors: MCSD_ERR_NULL, MCSD_ERR_BAD_SHAPE (B, N, V < 1, N > MCSD_MAX_NODES, B > 65535, R < 0 or R > 32,
 * n_roots or n_levels out of range), MCSD_ERR_WORKSPACE_TOO_SMALL, MCSD_ERR_CUDA.
 */
size_t mcsd_verify_tree_workspace_bytes(int B, int N, int V);

int mcsd_verify_tree(const float* p, const float* q,
                     const int32_t* tokens, const int32_t* parent, const int32_t* level_start,
                     int n_levels, int n_roots, const int32_t* gamma,
                     const float* u_accept, const float* u_bonus,
                     int B, int N, int V,
                     int32_t* accept_len, int32_t* out_tokens, int32_t* out_nodes,
                     int32_t* best_root, int32_t* next_roots, int R,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * mcsd_verify_tree from next-token logits (Fig. 1 step 4: the target's logits are turned into distributions;
 * Section 4.1: temperature 0.7 for probabilistic and 0 for greedy sampling).
 *
 *   temperature > 0   p = softmax(target_logits / temperature), q = softmax(draft_logits / temperature), then exactly
 *                     the procedure of mcsd_verify_tree.  p and q are formed on the fly from the logits (one extra
 *                     pass per visited node for the row maxima and normalisers) and never written to memory.
 *   temperature == 0  greedy: a candidate is accepted iff its token is the id of the largest target logit at its
 *                     parent (ties: lowest id; of several siblings with that token the first), the new token is
 *                     the largest target logit of the stop node, and next_roots lists the R largest target logits
 *                     there (ties: lower id first).  draft_logits, u_accept and u_bonus are not read and may be NULL.
 *
 *   target_logits, draft_logits   [dev] dtype[B][N][V]: row n holds the logits of the token that follows node n
 *   dtype                         MCSD_F32 or MCSD_BF16 (bf16 logits are widened to fp32 exactly)
 *   temperature                   0, or 1e-3 <= temperature <= 1e6
 *   all other arguments           as for mcsd_verify_tree; the workspace size is mcsd_verify_tree_workspace_bytes(B, N, V)
 *
 * Arithmetic: exponentials and row sums in fp32 per lane, fp64 across warps and for the acceptance ratio.
 * Errors: as mcsd_verify_tree, plus MCSD_ERR_BAD_DTYPE and MCSD_ERR_BAD_SHAPE for a temperature out of range.
 */
int mcsd_verify_tree_logits(const void* target_logits, const void* draft_logits, int dtype, float temperature,
                            const int32_t* tokens, const int32_t* parent, const int32_t* level_start,
                            int n_levels, int n_roots, const int32_t* gamma,
                            const float* u_accept, const float* u_bonus,
                            int B, int N, int V,
                            int32_t* accept_len, int32_t* out_tokens, int32_t* out_nodes,
                            int32_t* best_root, int32_t* next_roots, int R,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * Several new tokens for a target-initialised tree (Section 3.1: instead of one token, several are sampled from the
 * target side and become the roots of the next candidate tree).  To be called after mcsd_verify_tree (or
 * mcsd_verify_tree_logits with temperature > 0) on the same rows, results and workspace: for every sequence it draws
 * R distinct ids from the distribution the winning path stopped with -- the target row of the stop node, residualised
 * once per candidate rejected there -- one after the other: draw i is an inverse-CDF draw in token-id order with
 * uniform u_roots[b][i] over the ids not drawn before.  (The paper does not say how the tokens are drawn; distinct
 * tokens by sequential sampling without replacement is the reading taken here.  next_roots of mcsd_verify_tree
 * lists the most probable ids instead.)
 *
 *   p, q / target_logits, draft_logits, dtype, temperature   the rows given to the verify call
 *   accept_len, out_nodes, best_root   [dev] its results (out_nodes is [B][n_levels])
 *   u_roots        [dev] float[B][R] uniforms
 *   next_roots     [dev] int32[B][R] out; -1 where fewer than R ids carry mass
 *   workspace      [dev] the workspace the verify call used (read only here)
 *
 * One launch on `stream`.  Errors: MCSD_ERR_NULL, MCSD_ERR_BAD_SHAPE (sizes as for mcsd_verify_tree, R < 1 or R > 32,
 * temperature outside [1e-3, 1e6]), MCSD_ERR_BAD_DTYPE, MCSD_ERR_WORKSPACE_TOO_SMALL, MCSD_ERR_CUDA.
 */
int mcsd_sample_roots(const float* p, const float* q,
                      const int32_t* accept_len, const int32_t* out_nodes, const int32_t* best_root, int n_levels,
                      const float* u_roots, int B, int N, int V, int R, int32_t* next_roots,
                      const void* workspace, size_t workspace_bytes, void* stream);

int mcsd_sample_roots_logits(const void* target_logits, const void* draft_logits, int dtype, float temperature,
                             const int32_t* accept_len, const int32_t* out_nodes, const int32_t* best_root, int n_levels,
                             const float* u_roots, int B, int N, int V, int R, int32_t* next_roots,
                             const void* workspace, size_t workspace_bytes, void* stream);

/*
 * KV-cache update after acceptance (Fig. 1 step 6, where the accepted tokens join the sequence).  For every layer and
 * sequence b the keys/values of the winning root (node best_root[b]; with a single root that is node 0, the last
 * emitted token, which is not in the prefix cache yet) and of the accepted nodes out_nodes[b][0 .. accept_len[b]-1]
 * are copied from the tree tensors to cache rows seq_lens[b], seq_lens[b]+1, ..., then seq_lens[b] grows by
 * 1 + accept_len[b].  Rows that would fall beyond L_max are dropped and the length saturates at L_max.
 *
 *   k_cache_layers, v_cache_layers  [dev] arrays of n_layers device pointers, each a cache [B][H][L_max][D] (in/out)
 *   k_tree_layers, v_tree_layers    [dev] arrays of n_layers device pointers, each [B][H][N][D]
 *   seq_lens                        [dev] int32[B], in/out
 *   accept_len, out_nodes, best_root  [dev] outputs of mcsd_verify_tree (out_nodes is [B][n_levels])
 *   dtype                           MCSD_BF16 or MCSD_F32; D is 64 or 128; all tensors 16-byte aligned
 *
 * Two launches on `stream` for all layers together; no workspace.  Errors: MCSD_ERR_NULL, MCSD_ERR_BAD_SHAPE,
 * MCSD_ERR_BAD_DTYPE, MCSD_ERR_CUDA.
 */
int mcsd_commit_kv(void* const* k_cache_layers, void* const* v_cache_layers,
                   const void* const* k_tree_layers, const void* const* v_tree_layers, int n_layers,
                   int32_t* seq_lens, const int32_t* accept_len, const int32_t* out_nodes, const int32_t* best_root,
                   int n_levels, int B, int H, int N, int D, int L_max, int dtype, void* stream);

/*
 * mcsd_verify_tree with the vocabulary split over several GPUs (Fig. 1 steps 4-6, the procedure of
 * mcsd_verify_tree): rank r holds columns [v0, v0 + Vs) of p and q, the way a tensor-parallel output layer leaves
 * them, so no rank ever gathers a full row.  The four calls below are the per-rank kernels; between them the
 * caller reduces three small buffers over the ranks (with NCCL, or any all-reduce), in this order:
 *
 *   mcsd_verify_shard_gather                     -> all-reduce SUM of pq_exchange
 *   for round = 0 .. k:  mcsd_verify_shard_round -> all-reduce SUM of y_exchange   (not after round k)
 *   mcsd_verify_shard_select                     -> all-reduce SUM of mass_exchange
 *   mcsd_verify_shard_pick                       -> all-reduce MAX of out_tokens
 *
 * where k is the largest number of children of any node.  gather fetches p_u(x), q_u(x) of every candidate token
 * from the rank that owns x.  A round takes the reduced mass of the residual pass issued in the round before,
 * tests the next sibling of every undecided node and, on a rejection, adds up this rank's part of
 * sum_v max(p_v - c q_v, 0) for the next residual; decisions are recomputed alike on every rank from the reduced
 * numbers.  select follows the accepted paths (as mcsd_verify_tree) and reports this rank's share of the stop
 * distribution's mass; pick draws the new token by inverse CDF over the ranks' column ranges in order: the rank in
 * whose columns the running sum passes u_bonus * total writes the token, the others -1.  After the last
 * all-reduce every rank holds the outputs of mcsd_verify_tree (next_roots is not offered).
 *
 *   p_shard, q_shard  [dev] float[B][N][Vs], this rank's columns
 *   v0, V_total       first global token id of this rank's columns, size of the whole vocabulary; the ranks'
 *                     ranges are disjoint, in rank order, and cover [0, V_total)
 *   pq_exchange       [dev] double[B][N][2] (out of gather; read by round after the reduction)
 *   y_exchange        [dev] double[B][N] (in: reduced sums of the previous round; out: this rank's partial sums)
 *   mass_exchange     [dev] double[world][B][2] (out of select: row `rank` filled, others zero; read by pick)
 *   round             0 initialises the per-node state; rounds must be issued in order
 *   workspace         [dev] >= mcsd_verify_shard_workspace_bytes(B, N) bytes, the same one for all four calls
 *   tokens, parent, level_start, gamma, u_accept, u_bonus, accept_len, out_tokens, out_nodes, best_root:
 *                     as for mcsd_verify_tree, identical on every rank
 *
 * One launch per call on `stream`.  Errors: MCSD_ERR_NULL, MCSD_ERR_BAD_SHAPE (sizes as for mcsd_verify_tree with
 * Vs for V; v0 < 0 or v0 + Vs > V_total; rank outside [0, world); world > 1024; round outside [0, N]),
 * MCSD_ERR_WORKSPACE_TOO_SMALL, MCSD_ERR_CUDA.
 */
size_t mcsd_verify_shard_workspace_bytes(int B, int N);

int mcsd_verify_shard_gather(const float* p_shard, const float* q_shard, const int32_t* tokens,
                             const int32_t* parent, const int32_t* level_start, int n_levels,
                             const int32_t* gamma, int B, int N, int Vs, int v0, int V_total,
                             double* pq_exchange, void* stream);

int mcsd_verify_shard_round(const float* p_shard, const float* q_shard, const int32_t* parent,
                            const int32_t* level_start, int n_levels, const int32_t* gamma,
                            const float* u_accept, const double* pq_exchange, double* y_exchange,
                            int round, int B, int N, int Vs, void* workspace, size_t workspace_bytes,
                            void* stream);

int mcsd_verify_shard_select(const float* p_shard, const float* q_shard, const int32_t* tokens,
                             int n_levels, int n_roots, int B, int N, int Vs, int v0, int V_total,
                             int rank, int world, int32_t* accept_len, int32_t* out_tokens,
                             int32_t* out_nodes, int32_t* best_root, double* mass_exchange,
                             void* workspace, size_t workspace_bytes, void* stream);

int mcsd_verify_shard_pick(const float* p_shard, const float* q_shard, const float* u_bonus, int n_levels,
                           int B, int N, int Vs, int v0, int V_total, int rank, int world,
                           const double* mass_exchange, int32_t* out_tokens, const void* workspace,
                           size_t workspace_bytes, void* stream);

/*
 * mcsd_verify_tree with built-in scratch.  (The paper has no counterpart; this is a deployment convenience.)
 *
 * Same computation, arguments and results as mcsd_verify_tree, minus the workspace: the per-node scratch
 * lives in a fixed array inside the library image.  It is meant for callers that must not, or cannot,
 * obtain device memory at the point of the call: a serving engine that handed all of HBM to its KV-cache
 * pool at start-up so that a later cudaMalloc fails, a plug-in running under a host framework that owns the
 * allocator, or a latency-critical loop where an allocation's implicit synchronisation is not acceptable.
 * The call itself performs no cudaMalloc/cudaFree and calls no allocating library routine.
 *
 *   limit      B * N <= MCSD_STATIC_VERIFY_MAX_STATES, otherwise MCSD_ERR_STATIC_LIMIT is returned and
 *              nothing is launched.  The array costs about 320 KB on every GPU that loads the library, for
 *              the life of the process.
 *   first call The first call on each device looks up the array's device address (with that device
 *              current); make that first call outside any stream capture.
 *   sharing    All calls on one device use the same array, which still holds the previous call's contents;
 *              the entry point clears the part that has to start at zero.  Two calls that can overlap on the
 *              GPU (different streams, no dependency) race on it: order them, or use mcsd_verify_tree with
 *              separate workspaces.
 * Other errors: as mcsd_verify_tree.
 */
#define MCSD_STATIC_VERIFY_MAX_STATES 16384

int mcsd_verify_tree_static(const float* p, const float* q,
                            const int32_t* tokens, const int32_t* parent, const int32_t* level_start,
                            int n_levels, int n_roots, const int32_t* gamma,
                            const float* u_accept, const float* u_bonus,
                            int B, int N, int V,
                            int32_t* accept_len, int32_t* out_tokens, int32_t* out_nodes,
                            int32_t* best_root, int32_t* next_roots, int R,
                            void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MCSD_H_ */
