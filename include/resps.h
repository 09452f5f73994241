/*
 * resps.h -- C ABI of libresps: the per-step speculative-sampling hot path that
 * Re-SpS controls by re-choosing (TT, d, k) at every step.
 *
 * One speculative step is
 *   resps_tree_expand     draft-tree construction
 *   resps_tree_attention  tree-masked verification attention (once per layer)
 *   resps_verify_accept   per-node target argmax + longest accepted path
 *   resps_kv_compact      in-place KV-cache compaction of the accepted path
 *
 * General conventions
 *  - Every pointer named d_* or documented as DEVICE points to memory of the
 *    current CUDA device; every other pointer is HOST memory.
 *  - The caller owns every buffer it passes.  A context owns only its private
 *    device workspace (partial results, counters, a status word).
 *  - No hot call allocates, synchronises or reads device memory on the host:
 *    each only enqueues kernels on `stream`.  The per-step values (TT, d, k,
 *    prefix length, node counts) are read by the kernels from device memory,
 *    so they may change between calls -- or between replays of a captured CUDA
 *    graph -- without re-capture or recompilation.
 *  - A context serialises its workspace: calls on the same context must be
 *    ordered on one stream (or otherwise not overlap on the GPU).
 *  - Return value: RESPS_OK (0) or a negative RESPS_ERR_* code.  Argument
 *    errors are detected on the host before anything is enqueued.  Conditions
 *    only visible on the device (a step whose k exceeds the logits extent, a
 *    prefix that overruns the cache, ...) set bits in the context's device
 *    status word, which resps_status() copies back; the affected sequence is
 *    then processed with its parameters clamped into range.
 *  - Limits follow the paper's action space (Appendix A): TT <= 128, k <= 32,
 *    d <= 16.  TT, d, k are upper limits (the action space of Eq. 2): a tree
 *    has n = min(TT, 1 + k + (d-1) k^2) nodes, never an error.
 */
#ifndef RESPS_H_
#define RESPS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RESPS_MAX_TT 128
#define RESPS_MAX_K 32
#define RESPS_MAX_DEPTH 16
#define RESPS_STATIC_MAX_ROWS 1024 /* batch * max_tt limit of resps_target_argmax_static */

enum {
    RESPS_OK = 0,
    RESPS_ERR_INVALID_ARG = -1,       /* null pointer, non-positive size, misaligned buffer   */
    RESPS_ERR_UNSUPPORTED_SHAPE = -2, /* head_dim not 64/128, Hq % Hkv != 0, limits exceeded  */
    RESPS_ERR_CAPACITY = -3,          /* host-known: max_tt > kv_capacity, batch > max_batch  */
    RESPS_ERR_CUDA = -4,              /* a CUDA runtime call or launch failed                 */
    RESPS_ERR_NO_DEVICE = -5          /* no usable sm_100 device                              */
};

/* Bits of the device status word (resps_status). */
enum {
    RESPS_STATUS_STEP_CLAMPED = 1,   /* a step's tt/d/k was outside the supplied extents       */
    RESPS_STATUS_KV_OVERFLOW = 2,    /* prefix_len + n exceeds kv_capacity (the KV-cache       */
                                     /* overflow the paper's results section warns of); skipped */
    RESPS_STATUS_WAIT_TIMEOUT = 4,   /* a bounded device-side wait gave up                     */
    RESPS_STATUS_STALE_PLAN = 8      /* resps_tree_attention ran on a work list made for other  */
                                     /* step parameters (see resps_attention_replan)            */
};

typedef struct resps_ctx resps_ctx;      /* opaque */
typedef struct CUstream_st* resps_stream; /* a cudaStream_t */

/* Model shape and library limits, fixed per context. */
typedef struct {
    int32_t n_q_heads;  /* Hq                                               */
    int32_t n_kv_heads; /* Hkv, divides Hq                                  */
    int32_t head_dim;   /* D: 64 or 128                                     */
    int32_t vocab;      /* V                                                */
    int32_t max_batch;  /* sequences per call                               */
    int32_t max_tt;     /* <= RESPS_MAX_TT; row stride of all per-node arrays */
    int32_t max_k;      /* <= RESPS_MAX_K                                   */
    int32_t max_depth;  /* <= RESPS_MAX_DEPTH; retrieve / path rows hold max_depth+1 entries */
} resps_shape;

/* Per-sequence, per-step parameters (Eq. 2: the action (TT, d, k)); lives in DEVICE memory. */
typedef struct {
    int32_t tt;         /* total tree tokens including the root, >= 1       */
    int32_t d;          /* draft levels (node depths 1..d), >= 1            */
    int32_t k;          /* expansion top-k, 1 <= k <= min(V, max_k)         */
    int32_t prefix_len; /* L: tokens already in the KV cache                */
} resps_step;

/* Creates a context on the current device and allocates its workspace (the only
 * allocation the library performs).  Errors: INVALID_ARG, UNSUPPORTED_SHAPE,
 * NO_DEVICE, CUDA. */
int resps_create(resps_ctx** out, const resps_shape* shape);
/* Frees the workspace.  The caller must have synchronised all work using it. */
int resps_destroy(resps_ctx* ctx);
/* Static string for a return code. */
const char* resps_strerror(int code);
/* Synchronises `stream`, copies the device status word to *status and clears it.  After a
 * RESPS_STATUS_WAIT_TIMEOUT it also resets the workspace's arrival counters, so that the context
 * can serve further calls. */
int resps_status(resps_ctx* ctx, resps_stream stream, int32_t* status);
/* Bytes of device workspace held by the context. */
int64_t resps_workspace_bytes(const resps_ctx* ctx);

/*
 * Test and tuning aid, NOT part of the path: overrides one scheduling choice the library
 * otherwise makes by itself.  Results never depend on these values, only how the work is cut.
 * Returns INVALID_ARG for an unknown key.  (The paper has no counterpart.)
 */
enum {
    RESPS_DEBUG_ATTN_ROUNDS = 1,    /* rounds of work items the attention work list plans: 0 = its own choice */
    RESPS_DEBUG_ATTN_MIN_TILES = 2, /* fewest 64-key tiles a split of the keys is given (default 2)           */
    RESPS_DEBUG_ATTN_STAGGER = 3,   /* SM cycles the second half of a CTA starts behind the first (default 1000) */
    RESPS_DEBUG_SCAN_SLICES = 4,    /* slices a logits row is cut into by the streaming scan: 0 = its own choice */
    RESPS_DEBUG_ATTN_SINGLE = 5     /* single row tiles (both halves of a CTA on one tile) while no sequence has more
                                       than this many (row tiles per KV head)^2 x key tiles (default 2000)           */
};
int resps_debug_set(resps_ctx* ctx, int key, int value);

/*
 * Draft-tree construction (Section 3.2, "Draft Tree Expansion" and "Confidence-Based
 * Candidate Reranking"; Algorithm 2, tree-building loop and rerank).
 *
 * For every sequence b < batch, with (TT, d, k, L) = d_steps[b]:
 *   level 0: the k most probable tokens of row logits[b][0][0] become candidates 0..k-1
 *     (children of the root) with score log p;
 *   level j = 1..d-1: row logits[b][j][p] is the draft distribution after the p-th
 *     frontier node; its k most probable tokens become candidates
 *     c = k + (j-1) k^2 + p k + r with score = score(parent) + log p; the k best
 *     candidates of the level (score desc, candidate index asc) form the next frontier;
 *   rerank: the min(TT-1, n_cand) best of all candidates are kept and, in ascending
 *     candidate order, become nodes 1..n-1 behind the root (node 0).
 * Token order inside a row: value desc, token id asc.  log p = x - logsumexp(row).
 *
 * d_draft_logits  DEVICE fp32, element (b, level, slot, v) at
 *                 b*ld_b + level*ld_level + slot*ld_row + v; extents n_levels x n_slots
 *                 (level 0 uses slot 0 only).  16-byte aligned base and strides that are
 *                 multiples of 4 elements select the vectorised path.
 * d_root_token    DEVICE int32 [batch]
 * Outputs, DEVICE, row stride max_tt per sequence, entries >= n untouched:
 *   tokens, parent (root -1), depth, position_ids (= L + depth)   int32 [batch][max_tt]
 *   mask       uint64 [batch][max_tt][2]: bit j <=> node j is the node or an ancestor
 *   retrieve   int32 [batch][max_tt][max_depth+1]: one row per leaf in ascending leaf
 *              order, root-to-leaf node indices, -1 padded; rows >= n_leaves untouched
 *   n_leaves, n_nodes  int32 [batch]
 * A step with d > n_levels or k > n_slots (or k > V, or tt > max_tt) is clamped and
 * RESPS_STATUS_STEP_CLAMPED is set.
 */
int resps_tree_expand(resps_ctx* ctx, const resps_step* d_steps, int batch,
                      const float* d_draft_logits, int64_t ld_b, int64_t ld_level, int64_t ld_row,
                      int n_levels, int n_slots, const int32_t* d_root_token,
                      int32_t* d_tokens, int32_t* d_parent, int32_t* d_depth,
                      int32_t* d_position_ids, uint64_t* d_mask, int32_t* d_retrieve,
                      int32_t* d_n_leaves, int32_t* d_n_nodes, resps_stream stream);

/*
 * The same construction level by level, for a draft model that runs between levels (Section 3.2,
 * "Draft Tree Expansion": the k best tokens of a layer are expanded to the next layer; Algorithm 2:
 * the draft model is called inside the tree-building loop).
 *
 *   resps_tree_expand_begin(ctx, d_steps, batch, n_slots)
 *   for level j = 0 .. d-1:
 *       the draft model produces the rows of level j (level 0: one row, after the root; level j >= 1:
 *       one row per member of the frontier after level j-1, in slot order)
 *       resps_tree_expand_level(ctx, d_steps, batch, j, rows, ...)  ->  the frontier after level j
 *   resps_tree_expand_finish(ctx, d_steps, batch, d_root_token, <outputs of resps_tree_expand>)
 * yields exactly the tree resps_tree_expand builds from the same rows.  The number of levels given
 * bounds the depth (a step asking for more is clamped and flagged).
 *
 * d_level_logits  DEVICE fp32, element (b, slot, v) at b*ld_b + slot*ld_row + v
 * Frontier outputs, DEVICE, [batch][max_k], entries >= k untouched.  Member p of the frontier after
 * level j is "draft node" 1 + j k + p (the root is draft node 0): the order in which a draft model
 * appends its tokens' K/V behind the prefix.
 *   d_frontier_tokens         its token
 *   d_frontier_parent_slot    the slot of its parent in the frontier after level j-1 (-1: the root)
 *   d_frontier_position_ids   L + j + 1
 *   d_frontier_node_index     1 + j k + p
 *   d_frontier_mask   uint64 [batch][max_k][2]: ancestor-or-self bits over draft nodes, in the format
 *                     of resps_tree_attention (written as zero once 1 + (j+1) k exceeds 128 draft
 *                     nodes); with the rows collected level by level it lets the draft model run
 *                     resps_tree_attention over prefix + draft nodes
 *   d_frontier_score  fp64 [batch][max_k] or NULL: cumulative log-probability (log V_i)
 * Calls of one expansion must come in order on one stream; levels out of order return INVALID_ARG.
 */
int resps_tree_expand_begin(resps_ctx* ctx, const resps_step* d_steps, int batch, int n_slots);
int resps_tree_expand_level(resps_ctx* ctx, const resps_step* d_steps, int batch, int level,
                            const float* d_level_logits, int64_t ld_b, int64_t ld_row,
                            int32_t* d_frontier_tokens, int32_t* d_frontier_parent_slot,
                            int32_t* d_frontier_position_ids, int32_t* d_frontier_node_index,
                            uint64_t* d_frontier_mask, double* d_frontier_score, resps_stream stream);
int resps_tree_expand_finish(resps_ctx* ctx, const resps_step* d_steps, int batch, const int32_t* d_root_token,
                             int32_t* d_tokens, int32_t* d_parent, int32_t* d_depth, int32_t* d_position_ids,
                             uint64_t* d_mask, int32_t* d_retrieve, int32_t* d_n_leaves, int32_t* d_n_nodes,
                             resps_stream stream);

/*
 * Tree-masked verification attention for one layer (Section 3.2, "Verification Phase":
 * the target model scores all tree tokens in a single pass; Appendix D: attention masks
 * follow the tree).
 *
 * For sequence b with L = d_steps[b].prefix_len and n = d_n_nodes[b], node t < n, head h:
 *   O[t,h] = sum_j softmax_j(scale * q[t,h] . K[g,j]) V[g,j],   g = h / (Hq/Hkv),
 * over cache slots j in [0, L) and slots L+i for every set bit i of mask[b][t].
 * The tree tokens' K/V must already be stored at slots L .. L+n-1.  No other slot
 * influences the result.
 *
 * d_q, d_o     DEVICE bf16 [batch][max_tt][Hq][D]; rows >= n of d_o are never written, rows >= n of
 *              d_q may be read (whole tiles are fetched) but never influence a result
 * d_lse        DEVICE fp32 [batch][max_tt][Hq] or NULL: natural-log sum of exp of the scaled scores
 * d_k_cache, d_v_cache  DEVICE bf16; element (b, g, slot, e) at
 *              b*kv_stride_seq + g*kv_stride_head + slot*kv_stride_tok + e  (elements);
 *              16-byte aligned, strides multiples of 8 elements
 * kv_capacity  slots per (sequence, head), at most 2^21; a sequence with L + n > kv_capacity is
 *              skipped and RESPS_STATUS_KV_OVERFLOW set
 * softmax_scale  must be positive (INVALID_ARG otherwise)
 * d_mask       as written by resps_tree_expand
 * Accumulation is fp32; the result is rounded to bf16 once.
 *
 * How the work is cut over the GPU depends only on (d_steps, d_n_nodes), which are the same for
 * every layer of a step: the first call after resps_tree_expand (or after a resps_verify_accept
 * that advanced these d_steps, or resps_attention_replan) derives that work list on the device,
 * later calls with the same d_steps, d_n_nodes, batch, kv_capacity and stream reuse it.  A caller
 * that changes the contents of d_steps or d_n_nodes by other means between two calls must call
 * resps_attention_replan() in between; a call that finds its list out of date sets
 * RESPS_STATUS_STALE_PLAN (its results are then undefined).
 */
int resps_tree_attention(resps_ctx* ctx, const resps_step* d_steps, const int32_t* d_n_nodes,
                         int batch, const void* d_q, void* d_o, float* d_lse,
                         const void* d_k_cache, const void* d_v_cache, int64_t kv_stride_seq,
                         int64_t kv_stride_head, int64_t kv_stride_tok, int64_t kv_capacity,
                         const uint64_t* d_mask, float softmax_scale, resps_stream stream);

/* Host-only: the next resps_tree_attention call derives its work list anew (see there). */
int resps_attention_replan(resps_ctx* ctx);

/*
 * Greedy verification and acceptance (Section 3.1: greedy decoding; Section 3.2,
 * "Acceptance Criterion" at temperature 0 -- a draft token is accepted iff it equals the
 * target's argmax after its parent; Algorithm 2, "get accepted tokens").
 *
 * d_target_logits  DEVICE fp32, element (b, i, v) at b*ld_b + i*ld_row + v: the target
 *                  distribution after tree node i
 * d_tokens, d_parent  from resps_tree_expand
 * Outputs, DEVICE:
 *   d_target_argmax int32 [batch][max_tt]   argmax per node, ties -> lowest id
 *   d_accept_path   int32 [batch][max_depth+1]  node indices, path[0] = 0, unused -1
 *   d_accept_len    int32 [batch]           a = accepted draft tokens
 *   d_out_tokens    int32 [batch][max_depth+1]  the a accepted tokens then the bonus token
 *                                           (target argmax at the last accepted node), unused -1
 *   d_steps_next    resps_step [batch] or NULL: copy of d_steps with prefix_len += a+1.
 *                   It may alias d_steps (the step loop then advances on the device with no host
 *                   write); resps_kv_compact must in that case be told that the prefix lengths it
 *                   is given are the advanced ones (steps_advanced = 1).
 */
int resps_verify_accept(resps_ctx* ctx, const resps_step* d_steps, const int32_t* d_n_nodes,
                        int batch, const float* d_target_logits, int64_t ld_b, int64_t ld_row,
                        const int32_t* d_tokens, const int32_t* d_parent,
                        int32_t* d_target_argmax, int32_t* d_accept_path, int32_t* d_accept_len,
                        int32_t* d_out_tokens, resps_step* d_steps_next, resps_stream stream);

/*
 * Verification and acceptance under sampling, temperature T > 0 (Section 3.2, "Acceptance
 * Criterion": a draft token y is accepted with probability min(1, P_T(y|.) / P_d(y|.)); Section
 * 4.1, "Lossless Output Fidelity": speculative sampling with rejection-based correction keeps the
 * target model's output distribution).  The alternative to resps_verify_accept, which is the same
 * step at temperature 0.
 *
 * P_T(.|node i) = softmax(d_target_logits[b][i] / T); P_d(.|node i) = softmax(r / T) of the draft
 * row r the node's children were taken from.  From the root: the children of the current node
 * are tried in node order; child j with token x is accepted when u_accept < min(1, p(x) / q(x)) and
 * the walk moves on to it; after a rejection p becomes the normalised residual max(0, p - q) and q
 * loses x (renormalised), and the next sibling is tried against those.  When no child is accepted
 * (or the node has none) the step's last token is drawn from the current p by inverse CDF in token
 * order with u_sample.  For a chain this is the paper's rule; how siblings are tried is this
 * library's reading where the paper is silent.  All arithmetic is fp64.
 *
 * d_draft_logits  the same rows (and strides) resps_tree_expand was given for this tree.  Which row
 *                 stands behind which node is kept in the context by resps_tree_expand: call this
 *                 for the tree of the last resps_tree_expand on this context.
 * temperature     T > 0 (INVALID_ARG otherwise)
 * d_u_accept      DEVICE fp64 [batch][max_depth+1][max_k]: uniform (0,1) numbers, entry (level, j)
 *                 decides the j-th child tried at the walk's level `level`
 * d_u_sample      DEVICE fp64 [batch][max_depth+1]: entry `level` draws the token when the walk
 *                 stops at that level
 * Outputs as resps_verify_accept (no arg-max): d_accept_path, d_accept_len, d_out_tokens (the
 * accepted tokens, then the drawn one), d_steps_next (may alias d_steps, see there).
 */
int resps_verify_accept_sampled(resps_ctx* ctx, const resps_step* d_steps, const int32_t* d_n_nodes, int batch,
                                const float* d_target_logits, int64_t ld_b, int64_t ld_row,
                                const float* d_draft_logits, int64_t draft_ld_b, int64_t draft_ld_level,
                                int64_t draft_ld_row, float temperature, const int32_t* d_tokens,
                                const int32_t* d_parent, const double* d_u_accept, const double* d_u_sample,
                                int32_t* d_accept_path, int32_t* d_accept_len, int32_t* d_out_tokens,
                                resps_step* d_steps_next, resps_stream stream);

/*
 * In-place KV-cache compaction (Appendix D, "input update": rejected tokens are discarded
 * from the cache).  For every bound layer, KV head and j = 0..a:
 *   slot L+j  <-  slot L+path[j]     (K and V),   L = the prefix length before the step.
 * Slots beyond L+a are left as they are.
 *
 * d_steps         DEVICE resps_step [batch].  steps_advanced = 0: prefix_len is the step's own L.
 *                 steps_advanced = 1: the array was already advanced by resps_verify_accept
 *                 (d_steps_next aliased d_steps), i.e. prefix_len = L + a + 1, and L is recovered
 *                 from it and d_accept_len.
 * d_k_caches, d_v_caches  DEVICE arrays of n_layers DEVICE pointers (bf16 caches laid out as
 *                         in resps_tree_attention)
 * kv_capacity     slots per (sequence, head).  A sequence whose path would touch a slot outside
 *                 [0, kv_capacity) -- the sequence resps_tree_attention skipped for the same
 *                 reason -- or whose path holds an entry outside [0, max_tt) is left untouched and
 *                 RESPS_STATUS_KV_OVERFLOW set (the KV-cache overflow the paper's results section
 *                 warns of).
 */
int resps_kv_compact(resps_ctx* ctx, const resps_step* d_steps, int steps_advanced, int batch,
                     const int32_t* d_accept_path, const int32_t* d_accept_len,
                     void* const* d_k_caches, void* const* d_v_caches, int n_layers,
                     int64_t kv_stride_seq, int64_t kv_stride_head, int64_t kv_stride_tok,
                     int64_t kv_capacity, resps_stream stream);

/*
 * Controller glue: one call per decoding step, before resps_tree_expand (Algorithm 1, "Re-SpS with
 * Action Caching"; Eq. 4: the state s_t is the concatenation of three hidden layers of the target
 * model; Eq. 3 and Eq. 5: the reward is tokens per second, averaged over the cache interval; Appendix
 * A: the policy network has two hidden layers of 128 units over the filtered action grid).
 *
 * Per sequence b:
 *   - the step that has just finished (d_prev_accept_len, d_prev_elapsed_s; both NULL before the first
 *     step) adds (accepted + 1) / seconds to the open interval;
 *   - while the cached action is valid (0 < cache_step) it is kept and cache_step advances, wrapping to
 *     0 after `interval` steps;
 *   - at cache_step 0 the interval is closed (d_reward_avg[b] = mean reward of its steps, Eq. 5), the
 *     policy is evaluated on the state, logits = W3 tanh(W2 tanh(W1 s + b1) + b2) + b3, an action is
 *     chosen (temperature 0: arg-max, ties -> lowest index; else a draw from softmax(logits / T) by
 *     inverse CDF in action order with d_uniform[b]) and its (TT, d, k) written into d_steps[b].
 * The library reads (TT, d, k) from d_steps in device memory, so nothing else has to be told.
 *
 * policy          HOST struct of DEVICE pointers: fp32 weights, row-major [out][in]; actions int32
 *                 [n_actions][3] = (TT, d, k); n_features divisible by 3, hidden <= 256, n_actions <= 1024
 * d_hidden_h/m/l  DEVICE bf16 [batch][n_features / 3], row stride ld_hidden elements: the three layers'
 *                 hidden states, read where the model left them
 * d_state         DEVICE resps_controller_state [batch]; zero-initialised by the caller before the first step
 * d_logits        DEVICE fp32 [batch][n_actions] or NULL; d_action DEVICE int32 [batch] or NULL
 * The activation (tanh) and "accepted tokens = accepted drafts + 1" are this library's readings.
 */
typedef struct {
    const float *w1, *b1; /* [hidden][n_features], [hidden]   */
    const float *w2, *b2; /* [hidden][hidden], [hidden]       */
    const float *w3, *b3; /* [n_actions][hidden], [n_actions] */
    const int32_t* actions;
    int32_t n_features, hidden, n_actions;
} resps_policy;
typedef struct {
    int32_t cache_step;   /* position in the cache interval; 0: the policy is asked at this step */
    int32_t action;       /* cached action index (state starts zeroed: the first step asks anyway) */
    float reward_sum;     /* sum of tokens / second over the open interval */
    int32_t reward_steps;
} resps_controller_state;
int resps_controller_step(resps_ctx* ctx, const resps_policy* policy, const void* d_hidden_h,
                          const void* d_hidden_m, const void* d_hidden_l, int64_t ld_hidden, int batch,
                          int interval, float temperature, const double* d_uniform,
                          const int32_t* d_prev_accept_len, const float* d_prev_elapsed_s,
                          resps_controller_state* d_state, resps_step* d_steps, float* d_reward_avg,
                          float* d_logits, int32_t* d_action, resps_stream stream);

/*
 * Vocabulary sharded over several GPUs (Section 5: the 70B target model needs four GPUs; the paper does
 * not say how the work is split -- this is the split by vocabulary columns).  Rank p of P holds columns
 * [offset_p, offset_p + V_p) of every logits row and a context created with vocab = V_p (V_p >= max_k).
 * A step then is, on every rank:
 *   resps_row_scan_shard       the rank's columns of the draft rows -> k (value, local id) pairs and one
 *                              log-sum-exp per row
 *   (all-gather of those small arrays over the ranks: the caller's, e.g. NCCL)
 *   resps_tree_expand_merge    merges the P shards' rows (ids become global by d_shard_offset) and builds
 *                              the tree: identical on every rank, and identical to resps_tree_expand on
 *                              the whole rows
 *   resps_tree_attention       per rank on its own KV heads if the heads are sharded too (a context is
 *                              created with the rank's heads; nothing crosses between ranks)
 *   resps_target_argmax_shard  the rank's columns of the target rows -> one packed (value, local id) per node
 *   (all-gather)
 *   resps_verify_accept_merge  merges and walks: identical to resps_verify_accept on the whole rows
 * Row arrays are [batch][resps_scan_rows(ctx)][max_k] (values fp32, ids int32) and
 * [batch][resps_scan_rows(ctx)] (log-sum-exp, fp64); gathered arrays carry a leading [n_shards] dimension
 * (n_shards <= 16); keys are uint64 [batch][max_tt].  d_shard_offset: DEVICE int32 [n_shards].
 */
int64_t resps_scan_rows(const resps_ctx* ctx);
int resps_row_scan_shard(resps_ctx* ctx, const resps_step* d_steps, int batch, const float* d_draft_logits,
                         int64_t ld_b, int64_t ld_level, int64_t ld_row, int n_levels, int n_slots,
                         float* d_part_val, int32_t* d_part_id, double* d_part_lse, resps_stream stream);
int resps_tree_expand_merge(resps_ctx* ctx, const resps_step* d_steps, int batch, int n_levels, int n_slots,
                            int n_shards, const float* d_all_val, const int32_t* d_all_id, const double* d_all_lse,
                            const int32_t* d_shard_offset, const int32_t* d_root_token, int32_t* d_tokens,
                            int32_t* d_parent, int32_t* d_depth, int32_t* d_position_ids, uint64_t* d_mask,
                            int32_t* d_retrieve, int32_t* d_n_leaves, int32_t* d_n_nodes, resps_stream stream);
int resps_target_argmax_shard(resps_ctx* ctx, const int32_t* d_n_nodes, int batch, const float* d_target_logits,
                              int64_t ld_b, int64_t ld_row, uint64_t* d_part_key, resps_stream stream);
int resps_verify_accept_merge(resps_ctx* ctx, const resps_step* d_steps, const int32_t* d_n_nodes, int batch,
                              int n_shards, const uint64_t* d_all_key, const int32_t* d_shard_offset,
                              const int32_t* d_tokens, const int32_t* d_parent, int32_t* d_target_argmax,
                              int32_t* d_accept_path, int32_t* d_accept_len, int32_t* d_out_tokens,
                              resps_step* d_steps_next, resps_stream stream);

/*
 * Per-node target arg-max for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is the arg-max step of resps_verify_accept offered without a context.)
 *
 * resps_create() calls cudaMalloc for the workspace its kernels need.  Some callers cannot do
 * that: a serving process whose device memory was handed over whole to another allocator at
 * start-up (cudaMalloc then fails or fragments that pool), a plug-in that is only ever called
 * inside a region where allocation is forbidden, or code that runs after the memory budget of
 * the GPU has been frozen.  This entry point needs no context and allocates nothing -- no
 * cudaMalloc, no cudaFree, no allocating library call.  Its scratch (one packed partial result
 * per 8192-element piece of a row, and one arrival counter per row) lives in a fixed array
 * inside the library, 516 KB, which every GPU that loads the library holds until the process
 * exits.
 *
 *   d_n_nodes         DEVICE int32 [batch]: rows i < n_nodes[b] of sequence b are reduced
 *   d_target_logits   DEVICE fp32, element (b, i, v) at b*ld_b + i*ld_row + v
 *   d_target_argmax   DEVICE int32 [batch][max_tt]: arg-max per node, ties -> lowest id;
 *                     entries >= n_nodes[b] untouched
 * Results equal those resps_verify_accept writes to d_target_argmax.
 *
 * Limits and rules:
 *  - batch * max_tt <= RESPS_STATIC_MAX_ROWS (1024) and max_tt <= RESPS_MAX_TT; more returns
 *    RESPS_ERR_CAPACITY / RESPS_ERR_UNSUPPORTED_SHAPE before anything is enqueued.
 *  - The first call on each device looks up the array's device address (with that device
 *    current).  Make that first call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps what the last call left in it.
 *    Each call clears its counters on `stream` before the kernel runs, but two calls that can
 *    overlap on the GPU (different streams without an ordering between them) race on the
 *    array: order them.
 */
int resps_target_argmax_static(const int32_t* d_n_nodes, int batch, int max_tt, int vocab,
                               const float* d_target_logits, int64_t ld_b, int64_t ld_row,
                               int32_t* d_target_argmax, resps_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* RESPS_H_ */
