// Greedy acceptance walk and in-place KV-cache compaction.
//
// accept_walk_kernel (Section 3.2, "Acceptance Criterion" at temperature 0; Algorithm 2,
// "get accepted tokens"): from the root, follow the child whose token equals the target's
// argmax at the current node until no child matches.
//
// kv_compact_kernel (Appendix D, "input update": rejected tokens are discarded from the
// KV cache): slot L+j <- slot L+path[j] for j = 0..a, K and V, every KV head and layer.
#include "common.cuh"

namespace resps {
namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;

// One CTA of 128 threads per sequence: thread c owns tree node c.  (Used when the arg-max kernel
// could not take the walk along: rows that are not 16-byte aligned.)
__global__ void __launch_bounds__(RESPS_MAX_TT) accept_walk_kernel(const AcceptArgs a) {
    pdl_wait();  // the kernel before this one in the stream has completed
    pdl_launch_dependents();
    __shared__ int s_tgt[RESPS_MAX_TT];
    __shared__ int s_next[RESPS_MAX_DEPTH];
    accept_walk_device(a, blockIdx.x, threadIdx.x, s_tgt, s_next, false, [] { __syncthreads(); });
}

struct CompactArgs {
    const resps_step* steps;
    int steps_advanced;  // 1: steps[b].prefix_len already holds L + a + 1
    const int32_t *accept_path, *accept_len;
    void* const* k_caches;
    void* const* v_caches;
    int64_t stride_seq, stride_head, stride_tok, capacity;
    int n_kv_heads, head_dim, max_depth, max_tt;
    int32_t* status;
};

// One CTA per (K-or-V of a KV head, layer, sequence).  All source rows are read into
// registers before any destination row is written (a destination slot may be the source
// of an earlier path entry), so the move is safe in place.
__global__ void __launch_bounds__(128) kv_compact_kernel(const CompactArgs a) {
    pdl_wait();  // the kernel before this one in the stream has completed
    pdl_launch_dependents();
    const int b = blockIdx.z, layer = blockIdx.y;
    const int head = blockIdx.x >> 1, is_v = blockIdx.x & 1;
    const int cap = a.max_depth + 1;
    const int len = min(max(a.accept_len[b], 0), a.max_depth);
    const int L = max(a.steps[b].prefix_len - (a.steps_advanced ? len + 1 : 0), 0);
    // Every slot the move reads or writes must lie inside the cache, every path entry inside a tree.
    {
        int bad = 0;
        if (threadIdx.x <= len) {
            const int src = a.accept_path[b * cap + threadIdx.x];
            bad = (src < 0 || src >= a.max_tt || static_cast<int64_t>(L) + src >= a.capacity ||
                   static_cast<int64_t>(L) + threadIdx.x >= a.capacity);
        }
        if (__syncthreads_or(bad)) {
            if (threadIdx.x == 0 && blockIdx.x == 0 && layer == 0) atomicOr(a.status, RESPS_STATUS_KV_OVERFLOW);
            return;
        }
    }
    __nv_bfloat16* base = static_cast<__nv_bfloat16*>(is_v ? a.v_caches[layer] : a.k_caches[layer]) +
                          b * a.stride_seq + head * a.stride_head;
    const int vec_per_row = a.head_dim / 8;  // 16-byte pieces per row
    const int total = (len + 1) * vec_per_row;
    constexpr int kMaxPer = (RESPS_MAX_DEPTH + 1) * 16 / 128 + 1;
    uint4 regs[kMaxPer];
#pragma unroll
    for (int i = 0; i < kMaxPer; ++i) {
        const int idx = threadIdx.x + i * 128;
        if (idx < total) {
            const int j = idx / vec_per_row, e = idx % vec_per_row;
            const int src = a.accept_path[b * cap + j];
            regs[i] = *reinterpret_cast<const uint4*>(base + static_cast<int64_t>(L + src) * a.stride_tok + e * 8);
        }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kMaxPer; ++i) {
        const int idx = threadIdx.x + i * 128;
        if (idx < total) {
            const int j = idx / vec_per_row, e = idx % vec_per_row;
            *reinterpret_cast<uint4*>(base + static_cast<int64_t>(L + j) * a.stride_tok + e * 8) = regs[i];
        }
    }
}

}  // namespace

AcceptArgs make_accept_args(const resps_ctx* ctx, const resps_step* d_steps, const int32_t* d_n_nodes,
                            const int32_t* tokens, const int32_t* parent, const int32_t* target_argmax,
                            int32_t* accept_path, int32_t* accept_len, int32_t* out_tokens, resps_step* steps_next) {
    AcceptArgs a;
    a.steps = d_steps, a.n_nodes = d_n_nodes;
    a.tokens = tokens, a.parent = parent, a.target_argmax = target_argmax;
    a.max_tt = ctx->shape.max_tt, a.max_depth = ctx->shape.max_depth;
    a.accept_path = accept_path, a.accept_len = accept_len, a.out_tokens = out_tokens;
    a.steps_next = steps_next;
    return a;
}

cudaError_t launch_accept_walk(const resps_ctx* ctx, const resps_step* d_steps,
                               const int32_t* d_n_nodes, int batch, const int32_t* tokens,
                               const int32_t* parent, const int32_t* target_argmax,
                               int32_t* accept_path, int32_t* accept_len, int32_t* out_tokens,
                               resps_step* steps_next, cudaStream_t st) {
    const AcceptArgs a = make_accept_args(ctx, d_steps, d_n_nodes, tokens, parent, target_argmax, accept_path,
                                          accept_len, out_tokens, steps_next);
    return launch_pdl(accept_walk_kernel, dim3(batch), dim3(RESPS_MAX_TT), 0, st, a);
}

cudaError_t launch_kv_compact(const resps_ctx* ctx, const resps_step* d_steps, int steps_advanced, int batch,
                              const int32_t* accept_path, const int32_t* accept_len,
                              void* const* k_caches, void* const* v_caches, int n_layers,
                              int64_t stride_seq, int64_t stride_head, int64_t stride_tok,
                              int64_t capacity, cudaStream_t st) {
    CompactArgs a;
    a.steps = d_steps, a.steps_advanced = steps_advanced;
    a.accept_path = accept_path, a.accept_len = accept_len;
    a.k_caches = k_caches, a.v_caches = v_caches;
    a.stride_seq = stride_seq, a.stride_head = stride_head, a.stride_tok = stride_tok;
    a.capacity = capacity;
    a.n_kv_heads = ctx->shape.n_kv_heads, a.head_dim = ctx->shape.head_dim;
    a.max_depth = ctx->shape.max_depth, a.max_tt = ctx->shape.max_tt;
    a.status = ctx->ws.status;
    dim3 grid(ctx->shape.n_kv_heads * 2, n_layers, batch);
    return launch_pdl(kv_compact_kernel, grid, dim3(128), 0, st, a);
}

}  // namespace resps
