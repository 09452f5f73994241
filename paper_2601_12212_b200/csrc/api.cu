// C ABI of libresps: argument checks, the context and its workspace, and the
// sequencing of kernel launches behind each entry point (see include/resps.h).
#include <algorithm>
#include <cstring>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

namespace resps {
int scan_chunk_max();
int attention_item_rows();
int attention_max_rounds();
int attention_max_batch();
}  // namespace resps

namespace {

// A named range around the host side of an entry point (visible in a timeline tool when one is
// attached, free otherwise).  The names carry the component of the paper's time breakdown
// (Appendix C, Table 8) the call belongs to.
struct Range {
    explicit Range(const char* name) { nvtxRangePushA(name); }
    ~Range() { nvtxRangePop(); }
    Range(const Range&) = delete;
    Range& operator=(const Range&) = delete;
};

inline int64_t align_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

struct Carver {
    int64_t off = 0;
    char* base = nullptr;
    template <typename T>
    void take(T*& p, int64_t count) {
        off = align_up(off, 256);
        if (base) p = reinterpret_cast<T*>(base + off);
        off += count * static_cast<int64_t>(sizeof(T));
    }
};

void carve(resps_ctx* c, Carver& cv) {
    const resps_shape& s = c->shape;
    resps::Workspace& w = c->ws;
    const int64_t rows = static_cast<int64_t>(s.max_batch) * w.max_rows;
    const int64_t nodes = static_cast<int64_t>(s.max_batch) * s.max_tt;
    cv.take(w.status, 64);
    cv.take(w.row_counter, rows);
    cv.take(w.amax_counter, nodes);
    cv.take(w.amax_seq_counter, s.max_batch);
    cv.take(w.ctl_counter, s.max_batch);
    const int64_t zero_end = cv.off;  // everything above must start as zero
    (void)zero_end;
    cv.take(w.node_row, nodes);
    cv.take(w.amax_local, nodes);
    cv.take(w.ctl_h1, static_cast<int64_t>(s.max_batch) * resps::controller_max_hidden());
    cv.take(w.samp_scratch, static_cast<int64_t>(resps::sampled_scratch_doubles(s.max_batch, s.vocab)));
    cv.take(w.part_key, rows * w.scan_splits * s.max_k);
    cv.take(w.part_ms, rows * w.scan_splits);
    cv.take(w.row_val, rows * s.max_k);
    cv.take(w.row_id, rows * s.max_k);
    cv.take(w.row_lse, rows);
    cv.take(w.amax_part, nodes * w.scan_splits);
    cv.take(w.attn_plan, static_cast<int64_t>(resps::attention_plan_bytes(s.max_batch, w.attn_max_items)));
    cv.take(w.attn_part_o, static_cast<int64_t>(w.attn_max_items) * resps::attention_item_rows() * s.head_dim);
    cv.take(w.attn_part_ml, static_cast<int64_t>(w.attn_max_items) * resps::attention_item_rows());
}

#define RESPS_CHECK_PTR(p) \
    if ((p) == nullptr) return RESPS_ERR_INVALID_ARG

inline bool aligned16(const void* p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; }

}  // namespace

extern "C" {

const char* resps_strerror(int code) {
    switch (code) {
        case RESPS_OK: return "ok";
        case RESPS_ERR_INVALID_ARG: return "invalid argument";
        case RESPS_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case RESPS_ERR_CAPACITY: return "capacity exceeded";
        case RESPS_ERR_CUDA: return "CUDA error";
        case RESPS_ERR_NO_DEVICE: return "no usable sm_100 device";
        default: return "unknown error";
    }
}

int resps_create(resps_ctx** out, const resps_shape* shape) {
    RESPS_CHECK_PTR(out);
    RESPS_CHECK_PTR(shape);
    *out = nullptr;
    const resps_shape& s = *shape;
    if (s.n_q_heads < 1 || s.n_kv_heads < 1 || s.vocab < 1 || s.max_batch < 1 || s.max_tt < 1 ||
        s.max_k < 1 || s.max_depth < 1)
        return RESPS_ERR_INVALID_ARG;
    if ((s.head_dim != 64 && s.head_dim != 128) || s.n_q_heads % s.n_kv_heads != 0 ||
        s.max_tt > RESPS_MAX_TT || s.max_k > RESPS_MAX_K || s.max_depth > RESPS_MAX_DEPTH ||
        s.max_batch > resps::attention_max_batch())
        return RESPS_ERR_UNSUPPORTED_SHAPE;
    if (s.max_k + (s.max_depth - 1) * s.max_k * s.max_k > resps::tree_candidate_limit())
        return RESPS_ERR_UNSUPPORTED_SHAPE;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RESPS_ERR_NO_DEVICE;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return RESPS_ERR_NO_DEVICE;
    if (prop.major != 10) return RESPS_ERR_NO_DEVICE;

    resps_ctx* c = new (std::nothrow) resps_ctx();
    if (!c) return RESPS_ERR_CUDA;
    c->attn_host = nullptr;
    c->level_next = 0, c->level_slots = 1;
    c->shape = s;
    c->device = dev;
    c->sm_count = prop.multiProcessorCount;
    resps::Workspace& w = c->ws;
    // a scan CTA keeps its whole chunk in registers; up to 128 chunks per row (vocab <= 2^20)
    const int chunk = resps::scan_chunk_max();
    w.scan_chunk = chunk;
    w.scan_splits = (s.vocab + chunk - 1) / chunk;
    if (w.scan_splits > 128) {
        delete c;
        return RESPS_ERR_UNSUPPORTED_SHAPE;
    }
    w.max_rows = 1 + (s.max_depth - 1) * s.max_k;
    const int G = s.n_q_heads / s.n_kv_heads;
    const int item_rows = resps::attention_item_rows();
    w.attn_grid = c->sm_count;
    w.attn_min_tiles = 2;
    w.attn_max_groups = s.max_batch * s.n_kv_heads * ((s.max_tt * G + item_rows / 2 - 1) / (item_rows / 2));  // single row tiles
    w.attn_max_items = resps::attention_max_rounds() * w.attn_grid + w.attn_max_groups;

    Carver dry;
    carve(c, dry);
    c->arena_bytes = align_up(dry.off, 256);
    if (cudaMalloc(&c->arena, c->arena_bytes) != cudaSuccess) {
        delete c;
        return RESPS_ERR_CUDA;
    }
    if (cudaMemset(c->arena, 0, c->arena_bytes) != cudaSuccess) {
        cudaFree(c->arena);
        delete c;
        return RESPS_ERR_CUDA;
    }
    Carver real;
    real.base = static_cast<char*>(c->arena);
    carve(c, real);
    if (resps::attention_setup(c) != cudaSuccess || resps::tree_setup(c) != cudaSuccess ||
        resps::scan_setup(c) != cudaSuccess || resps::sampled_setup(c) != cudaSuccess) {
        cudaFree(c->arena);
        resps::attention_teardown(c);
        delete c;
        return RESPS_ERR_CUDA;
    }
    *out = c;
    return RESPS_OK;
}

int resps_destroy(resps_ctx* ctx) {
    if (!ctx) return RESPS_OK;
    cudaError_t e = cudaFree(ctx->arena);
    resps::attention_teardown(ctx);
    delete ctx;
    return e == cudaSuccess ? RESPS_OK : RESPS_ERR_CUDA;
}

int resps_attention_replan(resps_ctx* ctx) {
    RESPS_CHECK_PTR(ctx);
    resps::attention_plan_invalidate(ctx);
    return RESPS_OK;
}

int resps_debug_set(resps_ctx* ctx, int key, int value) {
    RESPS_CHECK_PTR(ctx);
    resps::Workspace& w = ctx->ws;
    switch (key) {
        case RESPS_DEBUG_ATTN_ROUNDS: w.attn_rounds = std::max(0, value); break;
        case RESPS_DEBUG_ATTN_MIN_TILES: w.attn_min_tiles = std::max(1, value); break;
        case RESPS_DEBUG_ATTN_SINGLE: w.attn_single = std::min(1 << 26, std::max(0, value)); break;
        case RESPS_DEBUG_ATTN_STAGGER: w.attn_stagger = std::min(100000, std::max(0, value)); break;
        case RESPS_DEBUG_SCAN_SLICES: w.scan_slices_hint = std::max(0, value); break;
#ifdef RESPS_WAIT_TEST
        case 100: w.test_drop = value; break;  // test build only: which copy is left out (see common.cuh)
#endif
        default: return RESPS_ERR_INVALID_ARG;
    }
    resps::attention_plan_invalidate(ctx);
    return RESPS_OK;
}

int64_t resps_workspace_bytes(const resps_ctx* ctx) { return ctx ? ctx->arena_bytes : 0; }

int resps_status(resps_ctx* ctx, resps_stream stream, int32_t* status) {
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(status);
    if (cudaMemcpyAsync(status, ctx->ws.status, sizeof(int32_t), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    if (cudaMemsetAsync(ctx->ws.status, 0, sizeof(int32_t), stream) != cudaSuccess) return RESPS_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return RESPS_ERR_CUDA;
    if (*status & RESPS_STATUS_WAIT_TIMEOUT) {
        // a kernel that gave up may have left arrival counters half-way: start them again from zero
        const resps::Workspace& w = ctx->ws;
        const size_t rows = static_cast<size_t>(ctx->shape.max_batch) * w.max_rows;
        const size_t nodes = static_cast<size_t>(ctx->shape.max_batch) * ctx->shape.max_tt;
        if (cudaMemsetAsync(w.row_counter, 0, rows * sizeof(unsigned int), stream) != cudaSuccess ||
            cudaMemsetAsync(w.amax_counter, 0, nodes * sizeof(unsigned int), stream) != cudaSuccess ||
            cudaMemsetAsync(w.amax_seq_counter, 0, ctx->shape.max_batch * sizeof(unsigned int), stream) != cudaSuccess ||
            cudaMemsetAsync(w.ctl_counter, 0, ctx->shape.max_batch * sizeof(unsigned int), stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess)
            return RESPS_ERR_CUDA;
    }
    return RESPS_OK;
}

int resps_tree_expand(resps_ctx* ctx, const resps_step* d_steps, int batch,
                      const float* d_draft_logits, int64_t ld_b, int64_t ld_level, int64_t ld_row,
                      int n_levels, int n_slots, const int32_t* d_root_token,
                      int32_t* d_tokens, int32_t* d_parent, int32_t* d_depth,
                      int32_t* d_position_ids, uint64_t* d_mask, int32_t* d_retrieve,
                      int32_t* d_n_leaves, int32_t* d_n_nodes, resps_stream stream) {
    Range range("resps_tree_expand [tree_construction]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(d_steps);
    RESPS_CHECK_PTR(d_draft_logits);
    RESPS_CHECK_PTR(d_root_token);
    RESPS_CHECK_PTR(d_tokens);
    RESPS_CHECK_PTR(d_parent);
    RESPS_CHECK_PTR(d_depth);
    RESPS_CHECK_PTR(d_position_ids);
    RESPS_CHECK_PTR(d_mask);
    RESPS_CHECK_PTR(d_retrieve);
    RESPS_CHECK_PTR(d_n_leaves);
    RESPS_CHECK_PTR(d_n_nodes);
    if (batch < 1 || n_levels < 1 || n_slots < 1 || ld_row < ctx->shape.vocab || ld_level < 0 || ld_b < 0)
        return RESPS_ERR_INVALID_ARG;
    if (batch > ctx->shape.max_batch) return RESPS_ERR_CAPACITY;
    if (n_levels > ctx->shape.max_depth) n_levels = ctx->shape.max_depth;
    if (n_slots > ctx->shape.max_k) n_slots = ctx->shape.max_k;
    resps::attention_plan_invalidate(ctx);  // a new tree: new node counts, possibly new step parameters
    if (resps::launch_row_scan(ctx, d_steps, batch, d_draft_logits, ld_b, ld_level, ld_row, n_levels,
                               n_slots, -1, stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    if (resps::launch_tree_build(ctx, d_steps, batch, n_levels, n_slots, d_root_token, d_tokens, d_parent,
                                 d_depth, d_position_ids, d_mask, d_retrieve, d_n_leaves, d_n_nodes,
                                 stream, true) != cudaSuccess)
        return RESPS_ERR_CUDA;
    return RESPS_OK;
}

// ---- vocabulary sharded over several GPUs -------------------------------------------------------------
int64_t resps_scan_rows(const resps_ctx* ctx) { return ctx ? ctx->ws.max_rows : 0; }

int resps_row_scan_shard(resps_ctx* ctx, const resps_step* d_steps, int batch, const float* d_draft_logits,
                         int64_t ld_b, int64_t ld_level, int64_t ld_row, int n_levels, int n_slots,
                         float* d_part_val, int32_t* d_part_id, double* d_part_lse, resps_stream stream) {
    Range range("resps_row_scan_shard [tree_construction]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(d_steps);
    RESPS_CHECK_PTR(d_draft_logits);
    RESPS_CHECK_PTR(d_part_val);
    RESPS_CHECK_PTR(d_part_id);
    RESPS_CHECK_PTR(d_part_lse);
    if (batch < 1 || n_levels < 1 || n_slots < 1 || ld_row < ctx->shape.vocab || ld_level < 0 || ld_b < 0)
        return RESPS_ERR_INVALID_ARG;
    if (batch > ctx->shape.max_batch) return RESPS_ERR_CAPACITY;
    if (ctx->shape.vocab < ctx->shape.max_k) return RESPS_ERR_UNSUPPORTED_SHAPE;  // a shard holds at least max_k columns
    if (n_levels > ctx->shape.max_depth) n_levels = ctx->shape.max_depth;
    if (n_slots > ctx->shape.max_k) n_slots = ctx->shape.max_k;
    if (resps::launch_row_scan(ctx, d_steps, batch, d_draft_logits, ld_b, ld_level, ld_row, n_levels, n_slots, -1,
                               stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    const resps::Workspace& w = ctx->ws;
    const size_t rows = static_cast<size_t>(batch) * w.max_rows;
    if (cudaMemcpyAsync(d_part_val, w.row_val, rows * ctx->shape.max_k * sizeof(float), cudaMemcpyDeviceToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(d_part_id, w.row_id, rows * ctx->shape.max_k * sizeof(int32_t), cudaMemcpyDeviceToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(d_part_lse, w.row_lse, rows * sizeof(double), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    return RESPS_OK;
}

int resps_tree_expand_merge(resps_ctx* ctx, const resps_step* d_steps, int batch, int n_levels, int n_slots,
                            int n_shards, const float* d_all_val, const int32_t* d_all_id, const double* d_all_lse,
                            const int32_t* d_shard_offset, const int32_t* d_root_token, int32_t* d_tokens,
                            int32_t* d_parent, int32_t* d_depth, int32_t* d_position_ids, uint64_t* d_mask,
                            int32_t* d_retrieve, int32_t* d_n_leaves, int32_t* d_n_nodes, resps_stream stream) {
    Range range("resps_tree_expand_merge [tree_construction]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(d_steps);
    RESPS_CHECK_PTR(d_all_val);
    RESPS_CHECK_PTR(d_all_id);
    RESPS_CHECK_PTR(d_all_lse);
    RESPS_CHECK_PTR(d_shard_offset);
    RESPS_CHECK_PTR(d_root_token);
    RESPS_CHECK_PTR(d_tokens);
    RESPS_CHECK_PTR(d_parent);
    RESPS_CHECK_PTR(d_depth);
    RESPS_CHECK_PTR(d_position_ids);
    RESPS_CHECK_PTR(d_mask);
    RESPS_CHECK_PTR(d_retrieve);
    RESPS_CHECK_PTR(d_n_leaves);
    RESPS_CHECK_PTR(d_n_nodes);
    if (batch < 1 || n_levels < 1 || n_slots < 1 || n_shards < 1) return RESPS_ERR_INVALID_ARG;
    if (n_shards > 16) return RESPS_ERR_UNSUPPORTED_SHAPE;
    if (batch > ctx->shape.max_batch) return RESPS_ERR_CAPACITY;
    if (n_levels > ctx->shape.max_depth) n_levels = ctx->shape.max_depth;
    if (n_slots > ctx->shape.max_k) n_slots = ctx->shape.max_k;
    resps::attention_plan_invalidate(ctx);
    if (resps::launch_shard_merge_rows(ctx, d_steps, batch, n_levels, n_slots, n_shards, d_all_val, d_all_id, d_all_lse,
                                       d_shard_offset, stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    if (resps::launch_tree_build(ctx, d_steps, batch, n_levels, n_slots, d_root_token, d_tokens, d_parent, d_depth,
                                 d_position_ids, d_mask, d_retrieve, d_n_leaves, d_n_nodes, stream, true) != cudaSuccess)
        return RESPS_ERR_CUDA;
    return RESPS_OK;
}

int resps_target_argmax_shard(resps_ctx* ctx, const int32_t* d_n_nodes, int batch, const float* d_target_logits,
                              int64_t ld_b, int64_t ld_row, uint64_t* d_part_key, resps_stream stream) {
    Range range("resps_target_argmax_shard [verification_process]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(d_n_nodes);
    RESPS_CHECK_PTR(d_target_logits);
    RESPS_CHECK_PTR(d_part_key);
    if (batch < 1 || ld_row < ctx->shape.vocab || ld_b < 0) return RESPS_ERR_INVALID_ARG;
    if (batch > ctx->shape.max_batch) return RESPS_ERR_CAPACITY;
    if (resps::launch_row_argmax(ctx, d_n_nodes, batch, d_target_logits, ld_b, ld_row, ctx->ws.amax_local, nullptr,
                                 nullptr, stream, reinterpret_cast<unsigned long long*>(d_part_key)) != cudaSuccess)
        return RESPS_ERR_CUDA;
    return RESPS_OK;
}

int resps_verify_accept_merge(resps_ctx* ctx, const resps_step* d_steps, const int32_t* d_n_nodes, int batch,
                              int n_shards, const uint64_t* d_all_key, const int32_t* d_shard_offset,
                              const int32_t* d_tokens, const int32_t* d_parent, int32_t* d_target_argmax,
                              int32_t* d_accept_path, int32_t* d_accept_len, int32_t* d_out_tokens,
                              resps_step* d_steps_next, resps_stream stream) {
    Range range("resps_verify_accept_merge [verification_process]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(d_steps);
    RESPS_CHECK_PTR(d_n_nodes);
    RESPS_CHECK_PTR(d_all_key);
    RESPS_CHECK_PTR(d_shard_offset);
    RESPS_CHECK_PTR(d_tokens);
    RESPS_CHECK_PTR(d_parent);
    RESPS_CHECK_PTR(d_target_argmax);
    RESPS_CHECK_PTR(d_accept_path);
    RESPS_CHECK_PTR(d_accept_len);
    RESPS_CHECK_PTR(d_out_tokens);
    if (batch < 1 || n_shards < 1) return RESPS_ERR_INVALID_ARG;
    if (batch > ctx->shape.max_batch) return RESPS_ERR_CAPACITY;
    if (d_steps_next) resps::attention_plan_invalidate(ctx, d_steps_next);
    if (resps::launch_shard_merge_argmax(ctx, d_n_nodes, batch, n_shards,
                                         reinterpret_cast<const unsigned long long*>(d_all_key), d_shard_offset,
                                         d_target_argmax, stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    if (resps::launch_accept_walk(ctx, d_steps, d_n_nodes, batch, d_tokens, d_parent, d_target_argmax, d_accept_path,
                                  d_accept_len, d_out_tokens, d_steps_next, stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    return RESPS_OK;
}

// ---- level form of the tree expansion --------------------------------------------------------------
int resps_tree_expand_begin(resps_ctx* ctx, const resps_step* d_steps, int batch, int n_slots) {
    Range range("resps_tree_expand_begin [tree_initialization]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(d_steps);
    if (batch < 1 || n_slots < 1) return RESPS_ERR_INVALID_ARG;
    if (batch > ctx->shape.max_batch) return RESPS_ERR_CAPACITY;
    ctx->level_next = 0;
    ctx->level_slots = n_slots > ctx->shape.max_k ? ctx->shape.max_k : n_slots;
    resps::attention_plan_invalidate(ctx);
    return RESPS_OK;
}

int resps_tree_expand_level(resps_ctx* ctx, const resps_step* d_steps, int batch, int level,
                            const float* d_level_logits, int64_t ld_b, int64_t ld_row,
                            int32_t* d_frontier_tokens, int32_t* d_frontier_parent_slot,
                            int32_t* d_frontier_position_ids, int32_t* d_frontier_node_index,
                            uint64_t* d_frontier_mask, double* d_frontier_score, resps_stream stream) {
    Range range("resps_tree_expand_level [drafting_process]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(d_steps);
    RESPS_CHECK_PTR(d_level_logits);
    RESPS_CHECK_PTR(d_frontier_tokens);
    RESPS_CHECK_PTR(d_frontier_parent_slot);
    RESPS_CHECK_PTR(d_frontier_position_ids);
    RESPS_CHECK_PTR(d_frontier_node_index);
    RESPS_CHECK_PTR(d_frontier_mask);
    if (batch < 1 || ld_row < ctx->shape.vocab || ld_b < 0 || level < 0) return RESPS_ERR_INVALID_ARG;
    if (batch > ctx->shape.max_batch) return RESPS_ERR_CAPACITY;
    if (level != ctx->level_next || level >= ctx->shape.max_depth) return RESPS_ERR_INVALID_ARG;  // levels come in order
    const int n_levels = ctx->shape.max_depth, n_slots = ctx->level_slots;
    if (resps::launch_row_scan(ctx, d_steps, batch, d_level_logits, ld_b, 0, ld_row, n_levels, n_slots, level,
                               stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    resps::FrontierOut out = {d_frontier_tokens, d_frontier_parent_slot, d_frontier_position_ids,
                              d_frontier_node_index, d_frontier_mask, d_frontier_score};
    if (resps::launch_tree_level(ctx, d_steps, batch, n_levels, n_slots, level, out, stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    ctx->level_next = level + 1;
    return RESPS_OK;
}

int resps_tree_expand_finish(resps_ctx* ctx, const resps_step* d_steps, int batch, const int32_t* d_root_token,
                             int32_t* d_tokens, int32_t* d_parent, int32_t* d_depth, int32_t* d_position_ids,
                             uint64_t* d_mask, int32_t* d_retrieve, int32_t* d_n_leaves, int32_t* d_n_nodes,
                             resps_stream stream) {
    Range range("resps_tree_expand_finish [tree_construction]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(d_steps);
    RESPS_CHECK_PTR(d_root_token);
    RESPS_CHECK_PTR(d_tokens);
    RESPS_CHECK_PTR(d_parent);
    RESPS_CHECK_PTR(d_depth);
    RESPS_CHECK_PTR(d_position_ids);
    RESPS_CHECK_PTR(d_mask);
    RESPS_CHECK_PTR(d_retrieve);
    RESPS_CHECK_PTR(d_n_leaves);
    RESPS_CHECK_PTR(d_n_nodes);
    if (batch < 1 || ctx->level_next < 1) return RESPS_ERR_INVALID_ARG;  // at least level 0 must have been given
    if (batch > ctx->shape.max_batch) return RESPS_ERR_CAPACITY;
    resps::attention_plan_invalidate(ctx);
    // the levels that were given bound the depth: a step asking for more is clamped (and flagged)
    if (resps::launch_tree_build(ctx, d_steps, batch, ctx->level_next, ctx->level_slots, d_root_token, d_tokens,
                                 d_parent, d_depth, d_position_ids, d_mask, d_retrieve, d_n_leaves, d_n_nodes,
                                 stream, false) != cudaSuccess)
        return RESPS_ERR_CUDA;
    ctx->level_next = 0;
    return RESPS_OK;
}

int resps_tree_attention(resps_ctx* ctx, const resps_step* d_steps, const int32_t* d_n_nodes,
                         int batch, const void* d_q, void* d_o, float* d_lse,
                         const void* d_k_cache, const void* d_v_cache, int64_t kv_stride_seq,
                         int64_t kv_stride_head, int64_t kv_stride_tok, int64_t kv_capacity,
                         const uint64_t* d_mask, float softmax_scale, resps_stream stream) {
    Range range("resps_tree_attention [target forward: tree attention]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(d_steps);
    RESPS_CHECK_PTR(d_n_nodes);
    RESPS_CHECK_PTR(d_q);
    RESPS_CHECK_PTR(d_o);
    RESPS_CHECK_PTR(d_k_cache);
    RESPS_CHECK_PTR(d_v_cache);
    RESPS_CHECK_PTR(d_mask);
    if (batch < 1 || kv_capacity < 1 || kv_stride_tok < ctx->shape.head_dim || kv_stride_head < 0 ||
        kv_stride_seq < 0 || !(softmax_scale > 0.f) || kv_capacity > (int64_t(1) << 21))
        return RESPS_ERR_INVALID_ARG;
    if (!aligned16(d_q) || !aligned16(d_o) || !aligned16(d_k_cache) || !aligned16(d_v_cache) ||
        kv_stride_seq % 8 || kv_stride_head % 8 || kv_stride_tok % 8)
        return RESPS_ERR_INVALID_ARG;
    if (batch > ctx->shape.max_batch || kv_capacity < ctx->shape.max_tt) return RESPS_ERR_CAPACITY;
    if (resps::launch_tree_attention(ctx, d_steps, d_n_nodes, batch, static_cast<const __nv_bfloat16*>(d_q),
                                     static_cast<__nv_bfloat16*>(d_o), d_lse,
                                     static_cast<const __nv_bfloat16*>(d_k_cache),
                                     static_cast<const __nv_bfloat16*>(d_v_cache), kv_stride_seq,
                                     kv_stride_head, kv_stride_tok, kv_capacity, d_mask, softmax_scale,
                                     stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    return RESPS_OK;
}

int resps_verify_accept(resps_ctx* ctx, const resps_step* d_steps, const int32_t* d_n_nodes,
                        int batch, const float* d_target_logits, int64_t ld_b, int64_t ld_row,
                        const int32_t* d_tokens, const int32_t* d_parent,
                        int32_t* d_target_argmax, int32_t* d_accept_path, int32_t* d_accept_len,
                        int32_t* d_out_tokens, resps_step* d_steps_next, resps_stream stream) {
    Range range("resps_verify_accept [verification_process]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(d_steps);
    RESPS_CHECK_PTR(d_n_nodes);
    RESPS_CHECK_PTR(d_target_logits);
    RESPS_CHECK_PTR(d_tokens);
    RESPS_CHECK_PTR(d_parent);
    RESPS_CHECK_PTR(d_target_argmax);
    RESPS_CHECK_PTR(d_accept_path);
    RESPS_CHECK_PTR(d_accept_len);
    RESPS_CHECK_PTR(d_out_tokens);
    if (batch < 1 || ld_row < ctx->shape.vocab || ld_b < 0) return RESPS_ERR_INVALID_ARG;
    if (batch > ctx->shape.max_batch) return RESPS_ERR_CAPACITY;
    if (d_steps_next) resps::attention_plan_invalidate(ctx, d_steps_next);  // prefix lengths move on
    // One kernel where the rows allow the streaming arg-max (the CTA that completes a sequence's last
    // row walks its tree); otherwise the walk is a second, small kernel.
    const resps::AcceptArgs walk = resps::make_accept_args(ctx, d_steps, d_n_nodes, d_tokens, d_parent, d_target_argmax,
                                                           d_accept_path, d_accept_len, d_out_tokens, d_steps_next);
    bool walked = false;
    if (resps::launch_row_argmax(ctx, d_n_nodes, batch, d_target_logits, ld_b, ld_row, d_target_argmax, &walk,
                                 &walked, stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    if (!walked && resps::launch_accept_walk(ctx, d_steps, d_n_nodes, batch, d_tokens, d_parent, d_target_argmax,
                                             d_accept_path, d_accept_len, d_out_tokens, d_steps_next,
                                             stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    return RESPS_OK;
}

int resps_verify_accept_sampled(resps_ctx* ctx, const resps_step* d_steps, const int32_t* d_n_nodes, int batch,
                                const float* d_target_logits, int64_t ld_b, int64_t ld_row,
                                const float* d_draft_logits, int64_t draft_ld_b, int64_t draft_ld_level,
                                int64_t draft_ld_row, float temperature, const int32_t* d_tokens,
                                const int32_t* d_parent, const double* d_u_accept, const double* d_u_sample,
                                int32_t* d_accept_path, int32_t* d_accept_len, int32_t* d_out_tokens,
                                resps_step* d_steps_next, resps_stream stream) {
    Range range("resps_verify_accept_sampled [verification_process]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(d_steps);
    RESPS_CHECK_PTR(d_n_nodes);
    RESPS_CHECK_PTR(d_target_logits);
    RESPS_CHECK_PTR(d_draft_logits);
    RESPS_CHECK_PTR(d_tokens);
    RESPS_CHECK_PTR(d_parent);
    RESPS_CHECK_PTR(d_u_accept);
    RESPS_CHECK_PTR(d_u_sample);
    RESPS_CHECK_PTR(d_accept_path);
    RESPS_CHECK_PTR(d_accept_len);
    RESPS_CHECK_PTR(d_out_tokens);
    if (batch < 1 || ld_row < ctx->shape.vocab || ld_b < 0 || draft_ld_row < ctx->shape.vocab || draft_ld_level < 0 ||
        draft_ld_b < 0 || !(temperature > 0.f))
        return RESPS_ERR_INVALID_ARG;
    if (batch > ctx->shape.max_batch) return RESPS_ERR_CAPACITY;
    if (d_steps_next) resps::attention_plan_invalidate(ctx, d_steps_next);  // prefix lengths move on
    if (resps::launch_accept_sampled(ctx, d_steps, d_n_nodes, batch, d_target_logits, ld_b, ld_row, d_draft_logits,
                                     draft_ld_b, draft_ld_level, draft_ld_row, static_cast<double>(temperature),
                                     d_tokens, d_parent, d_u_accept, d_u_sample, d_accept_path, d_accept_len,
                                     d_out_tokens, d_steps_next, stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    return RESPS_OK;
}

int resps_controller_step(resps_ctx* ctx, const resps_policy* policy, const void* d_hidden_h,
                          const void* d_hidden_m, const void* d_hidden_l, int64_t ld_hidden, int batch,
                          int interval, float temperature, const double* d_uniform,
                          const int32_t* d_prev_accept_len, const float* d_prev_elapsed_s,
                          resps_controller_state* d_state, resps_step* d_steps, float* d_reward_avg,
                          float* d_logits, int32_t* d_action, resps_stream stream) {
    Range range("resps_controller_step [rl_policy]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(policy);
    RESPS_CHECK_PTR(d_hidden_h);
    RESPS_CHECK_PTR(d_hidden_m);
    RESPS_CHECK_PTR(d_hidden_l);
    RESPS_CHECK_PTR(d_state);
    RESPS_CHECK_PTR(d_steps);
    RESPS_CHECK_PTR(d_reward_avg);
    RESPS_CHECK_PTR(policy->w1);
    RESPS_CHECK_PTR(policy->b1);
    RESPS_CHECK_PTR(policy->w2);
    RESPS_CHECK_PTR(policy->b2);
    RESPS_CHECK_PTR(policy->w3);
    RESPS_CHECK_PTR(policy->b3);
    RESPS_CHECK_PTR(policy->actions);
    if (batch < 1 || interval < 1 || policy->n_features < 3 || policy->n_features % 3 || policy->hidden < 1 ||
        policy->n_actions < 1 || ld_hidden < policy->n_features / 3 || temperature < 0.f ||
        (temperature > 0.f && !d_uniform) || ((d_prev_accept_len == nullptr) != (d_prev_elapsed_s == nullptr)))
        return RESPS_ERR_INVALID_ARG;
    if (policy->hidden > resps::controller_max_hidden() || policy->n_actions > resps::controller_max_actions())
        return RESPS_ERR_UNSUPPORTED_SHAPE;
    if (batch > ctx->shape.max_batch) return RESPS_ERR_CAPACITY;
    resps::attention_plan_invalidate(ctx, d_steps);  // (TT, d, k) may change
    if (resps::launch_controller(ctx, policy, d_hidden_h, d_hidden_m, d_hidden_l, ld_hidden, batch, interval,
                                 temperature, d_uniform, d_prev_accept_len, d_prev_elapsed_s, d_state, d_steps,
                                 d_reward_avg, d_logits, d_action, stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    return RESPS_OK;
}

int resps_kv_compact(resps_ctx* ctx, const resps_step* d_steps, int steps_advanced, int batch,
                     const int32_t* d_accept_path, const int32_t* d_accept_len,
                     void* const* d_k_caches, void* const* d_v_caches, int n_layers,
                     int64_t kv_stride_seq, int64_t kv_stride_head, int64_t kv_stride_tok,
                     int64_t kv_capacity, resps_stream stream) {
    Range range("resps_kv_compact [input_update]");
    RESPS_CHECK_PTR(ctx);
    RESPS_CHECK_PTR(d_steps);
    RESPS_CHECK_PTR(d_accept_path);
    RESPS_CHECK_PTR(d_accept_len);
    RESPS_CHECK_PTR(d_k_caches);
    RESPS_CHECK_PTR(d_v_caches);
    if (batch < 1 || n_layers < 1 || n_layers > 65535 || kv_stride_tok < ctx->shape.head_dim ||
        kv_stride_seq % 8 || kv_stride_head % 8 || kv_stride_tok % 8 || kv_capacity < 1 ||
        (steps_advanced != 0 && steps_advanced != 1))
        return RESPS_ERR_INVALID_ARG;
    if (batch > ctx->shape.max_batch) return RESPS_ERR_CAPACITY;
    if (resps::launch_kv_compact(ctx, d_steps, steps_advanced, batch, d_accept_path, d_accept_len, d_k_caches,
                                 d_v_caches, n_layers, kv_stride_seq, kv_stride_head, kv_stride_tok, kv_capacity,
                                 stream) != cudaSuccess)
        return RESPS_ERR_CUDA;
    return RESPS_OK;
}

}  // extern "C"
