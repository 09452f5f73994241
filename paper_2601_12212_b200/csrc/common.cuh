// Shared declarations of the libresps kernels (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "resps.h"

namespace resps {

// The test build (-DRESPS_WAIT_TEST, a separate library that only the bounded-wait test loads) gives
// every device-side wait a limit of about a millisecond and can leave out one copy, so that a wait
// really runs out; the product library is built without it.
#ifdef RESPS_WAIT_TEST
constexpr bool kWaitTest = true;
#else
constexpr bool kWaitTest = false;
#endif

constexpr int kScanThreads = 256;
constexpr int kWarp = 32;

// Host-side description of the context's device workspace.
struct Workspace {
    // vocabulary scans
    int scan_chunk = 0;       // elements of a row handled by one CTA
    int scan_splits = 0;      // ceil(V / scan_chunk)
    int scan_slices_hint = 0; // > 0: slices per row of the streaming scan (tuning aid)
    int max_rows = 0;         // 1 + (max_depth-1)*max_k
    unsigned long long* part_key = nullptr;  // [max_batch][max_rows][splits][max_k] packed (value,id)
    float2* part_ms = nullptr;               // [max_batch][max_rows][splits] (max, sum) in log2 domain
    unsigned int* row_counter = nullptr;     // [max_batch][max_rows]  arrival counters (self-resetting)
    float* row_val = nullptr;                // [max_batch][max_rows][max_k]
    int32_t* row_id = nullptr;               // [max_batch][max_rows][max_k]
    double* row_lse = nullptr;               // [max_batch][max_rows]
    unsigned long long* amax_part = nullptr; // [max_batch][max_tt][splits]
    unsigned int* amax_counter = nullptr;    // [max_batch][max_tt]
    int32_t* amax_local = nullptr;           // [max_batch][max_tt] shard-local arg-max ids (vocabulary sharding)
    int32_t* node_row = nullptr;             // [max_batch][max_tt] draft row behind every node's children (tree build)
    float* ctl_h1 = nullptr;                 // controller: first hidden layer [max_batch][256]
    unsigned int* ctl_counter = nullptr;     // controller: hidden units done per sequence (self-resetting)
    double* samp_scratch = nullptr;          // acceptance under sampling: partial sums, then (p, q) of every token and sequence
    unsigned int* amax_seq_counter = nullptr;  // [max_batch] arg-max CTAs of a sequence that have delivered (self-resetting)
    // attention
    int attn_grid = 0;          // persistent CTAs (one per SM)
    int attn_combine_flat_grid = 0;  // ... of its variant for batches
    int attn_min_tiles = 0;     // smallest key-tile count a split is given
    int attn_single = 2000;     // single row tiles while no sequence has more than this many row tiles^2 x key tiles
    int attn_stagger = 1000;    // cycles lane 1 starts behind lane 0 (RESPS_ATTN_STAGGER)
    int attn_rounds = 0;        // 0: chosen by the work list; else forced (RESPS_ATTN_ROUNDS, for tests)
    int attn_max_items = 0;     // partial slots
    unsigned char* attn_plan = nullptr;  // the attention work list: header, per-sequence and per-item entries
    __half* attn_part_o = nullptr;  // [items][item rows][D] fp16
    float4* attn_part_ml = nullptr; // [items][item rows]
    int attn_max_groups = 0;
    // Only read by the test build (RESPS_WAIT_TEST): bit 0 = the attention kernel's first V copy is
    // never issued, bit 1 = the streaming scan's second chunk copy is never issued.
    int test_drop = 0;
    // status
    int32_t* status = nullptr;
};

}  // namespace resps

struct resps_ctx {
    resps_shape shape;
    int device;
    int sm_count;
    void* arena;
    int64_t arena_bytes;
    resps::Workspace ws;
    int level_next, level_slots;  // level form of the tree expansion: the level expected next, the slots per level
    void* attn_host;  // host-side state of the attention launcher (tensor-map cache, work-list bookkeeping)
};

namespace resps {

// Arguments of the greedy acceptance walk (accept_walk_device below).
struct AcceptArgs {
    const resps_step* steps;
    const int32_t* n_nodes;
    const int32_t *tokens, *parent, *target_argmax;
    int max_tt, max_depth;
    int32_t *accept_path, *accept_len, *out_tokens;
    resps_step* steps_next;
};

// ---- launchers (one per translation unit) ---------------------------------
cudaError_t launch_row_scan(const resps_ctx* ctx, const resps_step* d_steps, int batch,
                            const float* logits, int64_t ld_b, int64_t ld_level, int64_t ld_row,
                            int n_levels, int n_slots, int only_level, cudaStream_t st);
// What the level form of the tree expansion hands back per level: the members of the new frontier.
struct FrontierOut {
    int32_t *tokens, *parent_slot, *position_ids, *node_index;  // [batch][max_k]
    uint64_t* mask;                                              // [batch][max_k][2]
    double* score;                                               // [batch][max_k] or null
};
cudaError_t launch_tree_level(const resps_ctx* ctx, const resps_step* d_steps, int batch, int n_levels, int n_slots,
                              int level, const FrontierOut& out, cudaStream_t st);
cudaError_t launch_tree_build(const resps_ctx* ctx, const resps_step* d_steps, int batch,
                              int n_levels, int n_slots, const int32_t* root_token,
                              int32_t* tokens, int32_t* parent, int32_t* depth, int32_t* position_ids,
                              uint64_t* mask, int32_t* retrieve, int32_t* n_leaves, int32_t* n_nodes,
                              cudaStream_t st, bool after_scan);  // after_scan: a scan or merge kernel of the same call precedes it
// Arg-max of every target row; with `walk` non-null and rows that allow the streaming kernel the
// acceptance walk runs in the same kernel (returns true through `walked`).
cudaError_t launch_row_argmax(const resps_ctx* ctx, const int32_t* d_n_nodes, int batch,
                              const float* logits, int64_t ld_b, int64_t ld_row, int32_t* argmax_out,
                              const AcceptArgs* walk, bool* walked, cudaStream_t st,
                              unsigned long long* key_out = nullptr);
cudaError_t launch_shard_merge_rows(const resps_ctx* ctx, const resps_step* d_steps, int batch, int n_levels, int n_slots,
                                    int n_shards, const float* all_val, const int32_t* all_id, const double* all_lse,
                                    const int32_t* shard_offset, cudaStream_t st);
cudaError_t launch_shard_merge_argmax(const resps_ctx* ctx, const int32_t* d_n_nodes, int batch, int n_shards,
                                      const unsigned long long* all_key, const int32_t* shard_offset, int32_t* out,
                                      cudaStream_t st);
AcceptArgs make_accept_args(const resps_ctx* ctx, const resps_step* d_steps, const int32_t* d_n_nodes,
                            const int32_t* tokens, const int32_t* parent, const int32_t* target_argmax,
                            int32_t* accept_path, int32_t* accept_len, int32_t* out_tokens, resps_step* steps_next);
cudaError_t launch_accept_walk(const resps_ctx* ctx, const resps_step* d_steps,
                               const int32_t* d_n_nodes, int batch, const int32_t* tokens,
                               const int32_t* parent, const int32_t* target_argmax,
                               int32_t* accept_path, int32_t* accept_len, int32_t* out_tokens,
                               resps_step* steps_next, cudaStream_t st);
cudaError_t launch_kv_compact(const resps_ctx* ctx, const resps_step* d_steps, int steps_advanced, int batch,
                              const int32_t* accept_path, const int32_t* accept_len,
                              void* const* k_caches, void* const* v_caches, int n_layers,
                              int64_t stride_seq, int64_t stride_head, int64_t stride_tok,
                              int64_t capacity, cudaStream_t st);
cudaError_t launch_tree_attention(const resps_ctx* ctx, const resps_step* d_steps,
                                  const int32_t* d_n_nodes, int batch, const __nv_bfloat16* q,
                                  __nv_bfloat16* o, float* lse, const __nv_bfloat16* k_cache,
                                  const __nv_bfloat16* v_cache, int64_t stride_seq,
                                  int64_t stride_head, int64_t stride_tok, int64_t capacity,
                                  const uint64_t* mask, float scale, cudaStream_t st);
cudaError_t attention_setup(resps_ctx* ctx);  // one-time function attributes, host-side state
void attention_teardown(resps_ctx* ctx);
// The arrays behind `steps_or_null` (step parameters or node counts; null = any) are about to change.
void attention_plan_invalidate(resps_ctx* ctx, const void* steps_or_null = nullptr);
size_t attention_plan_bytes(int max_batch, int max_items);

// Launch with programmatic stream serialization (see pdl_wait above).
template <typename Kernel, typename... Args>
cudaError_t launch_pdl(Kernel kernel, dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid, cfg.blockDim = block, cfg.dynamicSmemBytes = smem, cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr, cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}
cudaError_t launch_accept_sampled(const resps_ctx* ctx, const resps_step* d_steps, const int32_t* d_n_nodes, int batch,
                                  const float* target, int64_t ld_b, int64_t ld_row, const float* draft, int64_t dld_b,
                                  int64_t dld_level, int64_t dld_row, double temperature, const int32_t* tokens,
                                  const int32_t* parent, const double* u_accept, const double* u_sample,
                                  int32_t* accept_path, int32_t* accept_len, int32_t* out_tokens, resps_step* steps_next,
                                  cudaStream_t st);
size_t sampled_scratch_doubles(int max_batch, int vocab);
cudaError_t launch_controller(const resps_ctx* ctx, const resps_policy* pol, const void* h, const void* m, const void* l,
                              int64_t ld_hidden, int batch, int interval, float temperature, const double* uniform,
                              const int32_t* accept_len, const float* elapsed_s, resps_controller_state* state,
                              resps_step* steps, float* reward_avg, float* logits_out, int32_t* action_out,
                              cudaStream_t st);
int controller_max_hidden();
int controller_max_actions();
cudaError_t tree_setup(resps_ctx* ctx);
cudaError_t scan_setup(resps_ctx* ctx);
cudaError_t sampled_setup(resps_ctx* ctx);
int tree_candidate_limit();

// ---- device helpers --------------------------------------------------------
// Order-preserving map of a finite float onto uint32 (larger float -> larger key);
// -0 is folded onto +0 first so that equal floats give equal keys.
__device__ __forceinline__ uint32_t float_to_ordered(float f) {
    f = f + 0.0f;
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ordered_to_float(uint32_t k) {
    uint32_t u = (k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k;
    return __uint_as_float(u);
}
// Packed (value, id): a larger key ranks earlier under (value desc, id asc).
__device__ __forceinline__ unsigned long long pack_val_id(float v, int id) {
    return (static_cast<unsigned long long>(float_to_ordered(v)) << 32) |
           static_cast<unsigned long long>(0xFFFFFFFFu - static_cast<uint32_t>(id));
}
__device__ __forceinline__ float key_val(unsigned long long k) {
    return ordered_to_float(static_cast<uint32_t>(k >> 32));
}
__device__ __forceinline__ int key_id(unsigned long long k) {
    return static_cast<int>(0xFFFFFFFFu - static_cast<uint32_t>(k & 0xFFFFFFFFull));
}

// Programmatic dependent launch.  Every kernel of the library is launched so that it may start
// while its predecessor in the stream drains; it waits here before its first access to global
// memory and lets its own successor start right away (the successor waits in the same way, and
// the wait returns only when this grid has completed and flushed its writes).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Greedy acceptance walk (Section 3.2, "Acceptance Criterion" at temperature 0; Algorithm 2, "get
// accepted tokens"): from the root, follow the child whose token equals the target's arg-max at the
// current node until no child matches.  Run by `nthreads` >= RESPS_MAX_TT threads of one CTA for
// sequence b (thread c owns tree node c); `sync` is a barrier over exactly those threads.
// `s_tgt` [RESPS_MAX_TT] receives the targets' arg-max (the caller has filled it already when
// `have_targets`), `s_next` [RESPS_MAX_DEPTH] is scratch.  The hops are a chain of barriers over
// shared memory only: every global load is issued before the first hop, and the thread that owns
// the accepted node writes its entries itself.
template <typename Sync>
__device__ __forceinline__ void accept_walk_device(const AcceptArgs& a, int b, int tid, int* s_tgt, int* s_next,
                                                   bool have_targets, Sync sync) {
    const int n = min(max(a.n_nodes[b], 1), a.max_tt);
    const int64_t ob = static_cast<int64_t>(b) * a.max_tt;
    const int cap = a.max_depth + 1;
    const int my_tok = (tid < n) ? a.tokens[ob + tid] : -1;
    const int my_par = (tid < n) ? a.parent[ob + tid] : -2;
    resps_step step = {};
    if (tid == 0 && a.steps_next) step = a.steps[b];
    if (!have_targets && tid < n) s_tgt[tid] = __ldcg(a.target_argmax + ob + tid);
    if (tid < RESPS_MAX_DEPTH) s_next[tid] = -1;
    if (tid < cap) {
        a.accept_path[b * cap + tid] = (tid == 0) ? 0 : -1;
        a.out_tokens[b * cap + tid] = -1;
    }
    sync();  // (also orders the -1 fill above before the entries written below)
    int cur = 0, len = 0;
    for (int hop = 0; hop < a.max_depth; ++hop) {
        // children of one node carry distinct tokens, so at most one thread matches
        if (tid > 0 && tid < n && my_par == cur && my_tok == s_tgt[cur]) {
            s_next[hop] = tid;
            a.accept_path[b * cap + len + 1] = tid;
            a.out_tokens[b * cap + len] = my_tok;
        }
        sync();
        const int nxt = s_next[hop];
        if (nxt < 0) break;
        cur = nxt;
        ++len;
    }
    if (tid == 0) {
        a.out_tokens[b * cap + len] = s_tgt[cur];
        a.accept_len[b] = len;
        if (a.steps_next) {
            step.prefix_len += len + 1;
            a.steps_next[b] = step;
        }
    }
}

// Step parameters clamped into the extents the caller supplied.
struct StepDims {
    int tt, d, k, L;
    bool clamped;
};
__device__ __forceinline__ StepDims clamp_step(const resps_step& s, int n_levels, int n_slots,
                                                int max_tt, int max_k, int vocab) {
    StepDims r;
    r.tt = min(max(s.tt, 1), max_tt);
    r.d = min(max(s.d, 1), n_levels);
    int kmax = min(vocab, max_k);
    if (r.d > 1) kmax = min(kmax, n_slots);  // level 0 has a single row: slots bound k only beyond it
    r.k = min(max(s.k, 1), kmax);
    r.L = max(s.prefix_len, 0);
    r.clamped = (r.tt != s.tt) || (r.d != s.d) || (r.k != s.k) || (r.L != s.prefix_len);
    return r;
}

}  // namespace resps
