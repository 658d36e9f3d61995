/*
 * cast.h - C-ABI of the B200-native CAST hot path.
 *
 * One batched draft-and-verify step of cost-aware tree speculative decoding
 * (paper: "Inference-Cost-Aware Dynamic Tree Construction for Efficient
 * Inference in Large Language Models"):
 *
 *   cast_step_begin      root node, value 1                (Sec. "Tree Expansion Phase")
 *   cast_tree_expand     one draft layer: top-K children, path values,
 *                        breadth pruning (Eq. 1, Eq. 2, Algorithm 1),
 *                        depth pruning (Sec. "Dynamic Expansion Stage")
 *   cast_select_nodes    dynamic rerank (Sec. "Dynamic Reranking Stage"),
 *                        linearisation + ancestor mask (Sec. "Tree Reranking Phase")
 *   cast_tree_attention  verification attention under that mask
 *   cast_tree_attention_rows  the same for the rows of one layer of the growing tree (draft side)
 *   cast_accept          greedy acceptance (Sec. "Speculative Decoding", T = 0)
 *   cast_accept_stochastic  the same section's rule at T > 0, with residual resampling
 *   cast_compact_kv      accepted KV rows made contiguous
 *
 * Conventions
 *  - Plain C. Every tensor pointer is a DEVICE pointer owned by the caller
 *    unless its comment says "host". The library owns only what cast_create
 *    allocates (freed by cast_destroy).
 *  - `stream` is a cudaStream_t passed as void*. Compute calls only enqueue
 *    work: they never synchronise the host. Tree sizes (n_i, go/no-go, N) are
 *    decided on the device and stay there.
 *  - Compute calls allocate nothing. The split workspace of the attention is
 *    sized at set-up time by cast_reserve_attention; an attention call whose
 *    shape needs more than was reserved returns CAST_ERR_CAPACITY.
 *  - The return value reports errors the host can see (bad arguments, caps).
 *    Errors only the device can see (non-finite logits, a malformed tree, a
 *    page index out of range) are written to a device status word; read it with
 *    cast_poll_status, which synchronises `stream`.
 *  - cast_tree_expand, cast_select_nodes and cast_tree_attention are launched with programmatic
 *    dependent launch: their thread blocks may become resident while the previous kernel of the
 *    stream is still finishing, but they read no input (logits, Q, K/V, tree arrays, lengths) before
 *    that kernel has completed, so stream order keeps its usual meaning for the caller.
 *  - Precision of the tree-sizing decisions: node values, u, c and every comparison are fp64, but a row's
 *    log-sum-exp is accumulated in fp32 (about 3e-7 absolute per layer). The retained sets, n_i, go/stop
 *    and N equal those of an exact evaluation whenever no two neighbouring values across a kept/dropped
 *    boundary are closer than 1e-5 and no Algorithm 1 or depth test flips under a relative change of 2e-6
 *    of its two sides; closer than that, either outcome may be returned.
 *  - A context must not be used from two streams at once.
 *  - Row-major layouts, innermost index last, written as [d0, d1, ...].
 */
#ifndef CAST_H
#define CAST_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  CAST_OK = 0,
  CAST_ERR_INVALID_ARG = 1, /* null pointer, negative size, wrong call order          */
  CAST_ERR_SHAPE = 2,       /* head/group/dimension combination the kernels do not take */
  CAST_ERR_CAPACITY = 3,    /* a cap of this build or of the context is exceeded       */
  CAST_ERR_DTYPE = 4,
  CAST_ERR_COST_TABLE = 5,  /* no table for this batch size, or f not strictly increasing in n */
  CAST_ERR_BAD_TREE = 6,    /* device: parent[t] >= t, depth beyond max_depth, index out of range */
  CAST_ERR_BAD_PAGE = 7,    /* device: page-table entry out of range                     */
  CAST_ERR_NONFINITE = 8,   /* device: NaN or +inf logit, or a row without K finite logits */
  CAST_ERR_TIMEOUT = 9,     /* device: a bounded wait ran out                            */
  CAST_ERR_CUDA = 10        /* a CUDA runtime call failed                                */
} cast_status;

typedef enum { CAST_F32 = 0, CAST_BF16 = 1 } cast_dtype;

/* Caps of this build. */
#define CAST_MAX_TOP_K 16
#define CAST_MAX_WIDTH 16
#define CAST_MAX_DEPTH 16
#define CAST_MAX_TREE 128
#define CAST_MAX_BATCH 64

typedef struct cast_ctx cast_ctx;

#if defined(__GNUC__)
#define CAST_API __attribute__((visibility("default")))
#else
#define CAST_API
#endif

/*
 * Hyper-parameters (paper notation in brackets).
 *   top_k [K]        children generated per retained node, 1..CAST_MAX_TOP_K
 *   max_depth [H]    draft layers below the root = number of cast_tree_expand calls
 *   max_width [W]    most nodes retained per layer (0 means K); Algorithm 1 for
 *                    layer i runs on the first min(N_i, W, Ntab) sorted candidates
 *   max_tree [Ncap]  row stride of every per-tree-token array, <= CAST_MAX_TREE
 *   total_token [m]  cap on verified tokens, root included, <= max_tree
 *   C1, C2, C3       thresholds of breadth pruning, depth pruning, rerank
 *   fifo_len [R]     length of the depth-pruning buffers A_i
 *   enable_bp/dp/dr  breadth pruning / depth pruning / dynamic rerank. All three
 *                    off gives the fixed EAGLE-2 shape: n_i = min(K, N_i), all H
 *                    layers, N = min(pool, m).
 *   pool_mode        0: rerank over root + every generated candidate;
 *                    1: rerank over root + retained nodes only (N <= sum n_i)
 *   ctx_base_mode    0: context of Eq. 2 is sum_{j<i} n_j; 1: add n_0
 *   rerank_per_row   0: the rerank sizes the tree from the batch mean of the rank-wise values, as
 *                    Eq. 1 is printed: every sequence gets the same N. 1: every sequence runs the
 *                    rerank's Algorithm 1 on its own cumulative values (same cost row), so n_tree
 *                    differs per sequence; the per-layer sizing stays a batch decision (the next
 *                    draft forward is one rectangular batch). Needs enable_dr.
 */
typedef struct {
  double C1, C2, C3;
  int32_t max_batch, vocab, top_k, max_depth, max_width, max_tree, total_token;
  int32_t fifo_len, enable_bp, enable_dp, enable_dr, pool_mode, ctx_base_mode;
  int32_t rerank_per_row;
} cast_config;

/* Allocates the context and its device scratch on the current device.
 * Errors: INVALID_ARG, CAPACITY (a field beyond the caps above), CUDA. */
CAST_API cast_status cast_create(const cast_config* cfg, cast_ctx** out);
CAST_API cast_status cast_destroy(cast_ctx* ctx);
CAST_API const char* cast_status_string(cast_status s);

/*
 * Cost tables S_T(B), S_D(B) (Sec. "Method"): f(B, c, n) for c = g*L, g = 1..M and
 * n = 1..Ntab, as host arrays [M][Ntab] of doubles (copied; one pair per batch
 * size B, replacing an earlier pair for the same B). Synchronises the device.
 * Errors: COST_TABLE if a value is not finite and positive or a row is not
 * strictly increasing in n (precondition of Algorithm 1).
 */
CAST_API cast_status cast_set_cost_tables(cast_ctx* ctx, int B, int L, int M, int Ntab,
                                 const double* fT /* host */, const double* fD /* host */);

/*
 * Depth-pruning state (buffers A_1..A_{H-1}): the only state that outlives a
 * step. Blob layout: int32 H-1, int32 R, then for each buffer int32 count and R
 * doubles, oldest first. Call with blob = NULL to get the size. Both calls
 * synchronise the device.
 */
CAST_API cast_status cast_state_export(cast_ctx* ctx, void* blob /* host */, size_t* bytes);
CAST_API cast_status cast_state_import(cast_ctx* ctx, const void* blob /* host */, size_t bytes);

/*
 * Begin a step for B sequences: the pool of every row becomes {root}, root
 * value 1 (log-value 0), depth 0. root_token [B] int32: last accepted token.
 * kv_len [B] int32: prefix lengths; the padded context n_0 is their maximum.
 * Errors: CAPACITY (B > max_batch), COST_TABLE (a switch is on and B has no table).
 */
CAST_API cast_status cast_step_begin(cast_ctx* ctx, int B, const int32_t* root_token, const int32_t* kv_len,
                            void* stream);

/*
 * Expansion layer `layer` (1..H, in order). draft_logits [B, W, V]: row r of
 * sequence b is the draft distribution after the rank-r node retained by the
 * previous layer (layer 1: row 0 = root); rows >= n_{layer-1} are not read.
 * Children: the K tokens first in (logit descending, token id ascending); child
 * log-value = parent log-value + log-softmax. Then per sequence the N_i
 * candidates are sorted by (value desc, token asc, creation order), u (Eq. 1)
 * and c (Eq. 2) are formed, n_i = Algorithm 1(u, c, C1), and the depth test
 * Avg(A_i) * u_{n_i} / c_{n_i} >= C2 decides whether a further layer follows.
 * Outputs (device): next_tokens [B, W], next_parent_row [B, W] (which logits row
 * of this layer produced each retained node), -1 beyond n_i; next_count [1]:
 * n_i if a further layer follows, else 0 (layer H, or the depth test failed).
 * Once a layer was refused, later calls of the step only write next_count = 0.
 * -inf logits are legal (probability 0). Errors: INVALID_ARG when `layer` is
 * not the next layer of the step; device: NONFINITE.
 */
CAST_API cast_status cast_tree_expand(cast_ctx* ctx, int layer, const void* draft_logits, cast_dtype dtype,
                             int32_t* next_tokens, int32_t* next_parent_row, int32_t* next_count,
                             void* stream);

/*
 * Rerank and linearise. Pool nodes are sorted per sequence by (value desc,
 * depth asc, token asc, creation order); with v(s) the batch mean of the
 * rank-s values, u_k = sum_{s<=k} v(s), c_k = S_T[select(n_0)][k] / S_T[select(n_0)][1],
 * N = Algorithm 1(u, c, C3) capped by min(pool, m) (N = that cap if enable_dr = 0).
 * Each sequence keeps its own N best nodes, ordered by creation (root first,
 * parents before children). Outputs, all [B, Ncap] unless noted, entries >= N
 * are -1 (0 for anc_mask and scores):
 *   tokens, parent (linear index, -1 for the root), depth, pool_idx (int32);
 *   anc_mask [B, Ncap, ceil(Ncap/32)] uint32: bit j of row t set iff j is t or
 *   an ancestor of t; scores (double log-values; may be NULL); n_tree [B] int32.
 */
CAST_API cast_status cast_select_nodes(cast_ctx* ctx, int32_t* tokens, int32_t* parent, int32_t* depth,
                              uint32_t* anc_mask, int32_t* pool_idx, double* scores, int32_t* n_tree,
                              void* stream);

/*
 * Set-up call (synchronises the device and may allocate; not a compute call): sizes the context's
 * attention workspace for calls of cast_tree_attention / cast_tree_attention_rows with these arguments
 * (the partial results of the KV splits; nothing in the paper corresponds to it). The workspace only
 * grows: reserving several shapes keeps the largest. Every shape that will be used has to be reserved
 * once, before the first attention call of that shape and before any stream capture; an attention call
 * whose shape needs more than was reserved returns CAST_ERR_CAPACITY and launches nothing.
 * Errors: INVALID_ARG, DTYPE, SHAPE (as for cast_tree_attention), CAPACITY (B beyond max_batch), CUDA.
 */
CAST_API cast_status cast_reserve_attention(cast_ctx* ctx, cast_dtype dtype, int B, int Hq, int Hkv, int D,
                                   int page_size, int seq_capacity);

/*
 * Set-up call (nothing in the paper corresponds to it). The attention kernels are launched with programmatic
 * dependent launch and by default read nothing before the operation that precedes them on the stream has
 * completed. With promise != 0 the caller promises, for every later attention call of this context, that of the
 * call's inputs ONLY q and the cache rows of the tree tokens (positions >= kv_len[b]) can have been written by the
 * operation that immediately precedes the call on the stream; kv_len, n_tree, first_row, anc_mask, page_table and
 * the cache rows of the prefix (positions < kv_len[b]) were complete before that operation started (as they are in
 * a decoding loop: the tree is fixed for all layers of a step, and between two layers run the model's own kernels).
 * The kernel then decodes its work, reads the masks and fetches its first prefix tiles while its predecessor still
 * runs, and waits only before it loads q, a tile that reaches the tree tokens' rows, or writes output. It also
 * reuses, from one attention call to the next, the work list it decoded from kv_len, n_tree and the call's shape:
 * so the promise includes that kv_len, n_tree (and their pointers) keep their values between two attention calls
 * unless a call of this library changed them. Calls of this library that write those inputs (cast_select_nodes,
 * cast_compact_kv) or start a step (cast_step_begin) are accounted for by the library: the attention call that
 * follows one of them decodes afresh and takes no early reads. A caller that changes the lengths or tree sizes by
 * other means calls this function again (it discards the list). Needs bf16, D = 128 and a GQA group size that
 * divides 128; other shapes ignore the promise. promise = 0 (the default) restores the conservative behaviour.
 */
CAST_API cast_status cast_set_attention_early_reads(cast_ctx* ctx, int promise);

/*
 * One layer of verification attention (the mask of Sec. "Tree Reranking Phase"):
 * out[b,t,h] = softmax over {prefix positions 0..kv_len[b]-1} U {tree positions
 * kv_len[b]+j : bit j of anc_mask[b,t]} of (q . k) * scale, times v, for
 * t < n_tree[b]; rows t >= n_tree[b] of `out` are left untouched.
 * n_tree[b] must not exceed the context's total_token (device error BAD_TREE).
 *   q, out        [B, Ncap, Hq, D], dtype `dtype`; rows t >= n_tree[b] of q may hold anything (NaN and
 *                 inf included): they may be loaded with their neighbours but reach no output
 *   k_cache, v_cache  paged: [num_pages, page_size, Hkv, D]; the cache rows of
 *                 the tree tokens are already stored at positions kv_len[b]+j.
 *                 page_size = 0: contiguous [B, seq_capacity, Hkv, D].
 *   page_table    [B, seq_capacity] int32 page ids in [0, num_pages) (paged only;
 *                 seq_capacity is then the number of entries per sequence)
 *   scale         0 selects 1/sqrt(D)
 * Accumulation is fp32. Needs Hq % Hkv == 0, D in {64, 128}, 16-byte aligned
 * pointers, and a workspace reserved for this shape (cast_reserve_attention; else CAST_ERR_CAPACITY).
 * Device errors: BAD_PAGE.
 */
CAST_API cast_status cast_tree_attention(cast_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                                cast_dtype dtype, int B, int Hq, int Hkv, int D, int page_size,
                                const int32_t* page_table, int seq_capacity, int num_pages,
                                const int32_t* kv_len, const uint32_t* anc_mask, const int32_t* n_tree,
                                float scale, void* out, void* stream);

/*
 * cast_tree_attention restricted to the output rows t >= first_row[b] of every sequence: the tree
 * tokens before first_row[b] serve as context only (their K/V rows in the cache and their bits in
 * the masks are used, their queries are not read and their output rows are left untouched). This
 * is the draft model's attention while the tree grows (Sec. "Tree Expansion Phase"; Eq. 2 names its
 * context sum_{j<i} n_j): the linear order of a tree is creation order, so the tree after layer i is
 * a prefix of the final one; with n_tree[b] = tokens up to and including layer i and first_row[b] =
 * tokens before layer i the call computes layer i's n_i query rows against the prefix and the earlier
 * layers. first_row [B] device int32 (clamped to [0, n_tree[b]]); NULL means 0 everywhere, which is
 * cast_tree_attention. All other arguments, layouts and errors as for cast_tree_attention.
 */
CAST_API cast_status cast_tree_attention_rows(cast_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                                     cast_dtype dtype, int B, int Hq, int Hkv, int D, int page_size,
                                     const int32_t* page_table, int seq_capacity, int num_pages,
                                     const int32_t* kv_len, const uint32_t* anc_mask, const int32_t* n_tree,
                                     const int32_t* first_row, float scale, void* out, void* stream);

/*
 * Greedy acceptance: g[t] = argmax of target_logits[b,t,:] (ties: lower id).
 * Starting at the root, step to the child c of the current node with
 * tokens[c] == g[current] (lowest index if several) until there is none.
 *   target_logits [B, Ncap, V]; tokens, parent [B, Ncap]; n_tree [B]
 *   accept_len [B]   drafts accepted (root excluded)
 *   accept_path [B, H+1]  linear tree indices, root first, -1 padded
 *   bonus_token [B]  g at the last accepted node
 * `depth` and `anc_mask` may be NULL (not needed by the walk).
 * n_tree[b] must not exceed the context's total_token: only that many rows per sequence are swept.
 * Device errors: BAD_TREE (n_tree[b] < 1 or beyond total_token: the sequence gets accept_len 0, bonus 0 and a
 * path of -1; parent[t] >= t; a path longer than H+1).
 */
CAST_API cast_status cast_accept(cast_ctx* ctx, const void* target_logits, cast_dtype dtype, int B,
                        const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                        const uint32_t* anc_mask, const int32_t* n_tree, int32_t* accept_len,
                        int32_t* accept_path, int32_t* bonus_token, void* stream);

/*
 * Acceptance at temperature T > 0 (Sec. "Speculative Decoding"): a draft token x with draft
 * probability q = P_D(x | .) and target probability p = P_T(x | .) is accepted iff
 * u <= min(1, p / q); after a rejection the target distribution is replaced by the residual
 * norm(max(0, P_T - P_D)). On the tree: starting at the root, the children of the current node are
 * tried in tree order (ascending linear index), each against the distribution its rejected elder
 * siblings left (P_D unchanged); the first accepted child becomes the current node. When no child
 * is accepted (or there is none) the bonus token is drawn from the distribution that stands then -
 * P_T at a leaf, a residual otherwise - by inversion of its cumulative sum in token order: the
 * first token whose cumulative sum reaches u_bonus * total. A residual that sums to zero ends the
 * sibling loop with the distribution before it. Both distributions are softmax(logits / temperature).
 *   target_logits [B, Ncap, V]  row t: the target model's logits at tree token t
 *   draft_logits  [B, Ncap, V]  row t: the draft model's logits at tree token t, i.e. the
 *                               distribution t's children were drawn from; rows of leaves are not read
 *   temperature   > 0 (host)
 *   tokens, parent [B, Ncap]; n_tree [B]
 *   u_accept [B, Ncap] fp64 in (0,1): the uniform number of tree token t (root's entry unused)
 *   u_bonus  [B]       fp64 in (0,1)
 *   accept_len, accept_path, bonus_token: as for cast_accept
 * The random numbers are inputs so that the step is reproducible; the caller draws them.
 * All arithmetic is fp64. One thread-block cluster per sequence; the launch reads only the rows of
 * the nodes on the accepted path.
 * Device errors: BAD_TREE (n_tree out of range, a token outside [0, V), a path longer than H+1),
 * NONFINITE (a row whose exponentials do not sum to a positive finite number).
 */
CAST_API cast_status cast_accept_stochastic(cast_ctx* ctx, const void* target_logits, const void* draft_logits,
                                            cast_dtype dtype, int B, double temperature, const int32_t* tokens,
                                            const int32_t* parent, const int32_t* n_tree, const double* u_accept,
                                            const double* u_bonus, int32_t* accept_len, int32_t* accept_path,
                                            int32_t* bonus_token, void* stream);

/*
 * How cast_accept_stochastic organises its launch for this context's vocabulary and a logits dtype
 * (host-side query; no device work): the thread-block cluster size per sequence (16 where the
 * device can co-schedule that many CTAs with their shared memory, else 8, else 1) and whether a
 * CTA's vocabulary slice fits in shared memory (1) or every sweep recomputes it from the logits (0).
 * cast_accept_stochastic makes this query itself on its first call; call it before a stream capture.
 */
CAST_API cast_status cast_accept_stochastic_plan(cast_ctx* ctx, cast_dtype dtype, int* cluster_size /* host */,
                                                 int* cached /* host */);

/*
 * KV compaction (not in the paper; the plain gather): for every layer, kv-head
 * and j = 0..accept_len[b], cache row kv_len[b]+j := old row kv_len[b]+accept_path[b,j],
 * K and V, with out-of-place semantics; then kv_len[b] += accept_len[b] + 1.
 * Layer l of a cache starts layer_stride_bytes * l after the base pointer.
 * Cache layout, page_size, page_table, seq_capacity, num_pages as for
 * cast_tree_attention. Device errors: BAD_PAGE (also for a path entry < 0 or below its own place on the path,
 * or a row past the sequence's capacity: nothing is stored and kv_len stays).
 */
CAST_API cast_status cast_compact_kv(cast_ctx* ctx, void* k_cache, void* v_cache, cast_dtype dtype, int B,
                            int n_layers, size_t layer_stride_bytes, int Hkv, int D, int page_size,
                            const int32_t* page_table, int seq_capacity, int num_pages,
                            const int32_t* accept_path, const int32_t* accept_len,
                            int32_t* kv_len /* in/out */, void* stream);

/*
 * cast_accept for callers that must not allocate device memory. (The paper has no counterpart:
 * this entry point exists for hosts of the library, not for the method.)
 *
 * Some callers cannot call cudaMalloc at the point where they need the acceptance step: code that
 * runs inside a memory-pool or arena discipline where every device byte is accounted for up front,
 * code that runs after start-up in a process whose allocator has been frozen, or a plug-in that is
 * handed device pointers but no allocator. cast_accept needs a context, and a context allocates.
 * This variant takes no context and allocates nothing: the only scratch it needs (the per-chunk
 * winners of the target argmax sweep) lives in a fixed 512 KB array inside the library image, which
 * every GPU that loads the library holds until the process exits.
 *
 * Arguments as for cast_accept, with the sizes a context would carry passed explicitly: n_cap (row
 * stride of tokens/parent and of the logits' second axis, <= CAST_MAX_TREE), vocab, max_depth
 * (accept_path has max_depth + 1 entries per sequence). Limit: B * n_cap <= 2048, else
 * CAST_ERR_CAPACITY. There is no device status word: a malformed tree ends the walk early instead
 * of being reported.
 *
 * The first call on a device looks up the array's device address (no allocation, but a runtime
 * query): make that call before any stream capture. All calls share the one array, which keeps
 * the previous call's contents; a call overwrites every entry it later reads, so nothing needs
 * clearing, but two calls that overlap on the GPU (different streams) race on it.
 */
CAST_API cast_status cast_accept_static(const void* target_logits, cast_dtype dtype, int B, int n_cap, int vocab,
                                        int max_depth, const int32_t* tokens, const int32_t* parent,
                                        const int32_t* n_tree, int32_t* accept_len, int32_t* accept_path,
                                        int32_t* bonus_token, void* stream);

/* Synchronises `stream`, returns the device status word and clears it.
 * detail: an index that identifies the offending row/entry (meaning per status). */
CAST_API cast_status cast_poll_status(cast_ctx* ctx, void* stream, cast_status* device_status, int32_t* detail);

/*
 * Synchronises `stream` and copies the step counters to host int32 info[4 + H]:
 * info[0] layers generated, info[1] pool size, info[2] n_0, info[3] N of the
 * last cast_select_nodes (0 before), info[4 + i - 1] = n_i.
 */
CAST_API cast_status cast_step_info(cast_ctx* ctx, void* stream, int32_t* info /* host */);

#ifdef __cplusplus
}
#endif
#endif /* CAST_H */
