// Draft-tree build from the scanned rows (Section 3.2, "Draft Tree Expansion":
// cumulative score V_i along the root path, the k best of a layer are expanded;
// "Confidence-Based Candidate Reranking": all expanded tokens are reranked and the
// best TT-1 kept; Algorithm 2, tree-building loop).  One CTA per sequence; integer
// and fp64 work on at most k + (d-1)k^2 candidates, all in shared memory.
//
// A candidate's rank inside its level (at most k^2 candidates) is found by counting;
// its rank in the global rerank is its level rank plus binary searches over the
// other levels' sorted orders, and only the first TT-1 of a level can be kept at all.
#include <cmath>

#include "common.cuh"

namespace resps {
namespace {

constexpr int kTreeThreads = 1024;
constexpr unsigned kFull = 0xFFFFFFFFu;

struct TreeArgs {
    const resps_step* steps;
    int n_levels, n_slots;
    int vocab, max_tt, max_k, max_depth, max_rows;
    const float* row_val;
    const int32_t* row_id;
    const double* row_lse;
    const int32_t* root_token;
    int32_t *tokens, *parent, *depth, *position_ids;
    uint64_t* mask;
    int32_t *retrieve, *n_leaves, *n_nodes;
    int32_t* node_row;  // workspace [batch][max_tt]: level * RESPS_MAX_K + slot of the draft row a node's children came from
    int32_t* status;
    int cand_cap;  // candidates the shared-memory arrays hold
    // Level form: emit_level = j >= 0 ranks the levels up to j from the rows scanned so far, hands out
    // the frontier after level j and stops; -1 builds the whole tree.
    int emit_level;
    FrontierOut fr;
};

// Candidate order of the method: larger score first, equal scores by lower index.
__device__ __forceinline__ bool before(double sa, int ca, double sb, int cb) {
    return (sa > sb) || (sa == sb && ca < cb);
}

// Entries of the sorted index list `lst[0..n)` that rank before candidate (s, c).
__device__ __forceinline__ int count_before(const int* lst, int n, const double* score, double s, int c) {
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        const int e = lst[mid];
        if (before(score[e], e, s, c))
            lo = mid + 1;
        else
            hi = mid;
    }
    return lo;
}

// Exclusive prefix sum of one int per thread over the CTA; returns the total via `total`.
__device__ __forceinline__ int block_exclusive_scan(int v, int* s_warp, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = (lane < kTreeThreads / 32) ? s_warp[lane] : 0;
        int winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(kFull, winc, o);
            if (lane >= o) winc += t;
        }
        s_warp[lane] = winc - w;
        if (lane == 31) s_warp[32] = winc;
    }
    __syncthreads();
    total = s_warp[32];
    const int r = s_warp[warp] + inc - v;
    __syncthreads();
    return r;
}

__global__ void __launch_bounds__(kTreeThreads, 1) tree_build_kernel(const TreeArgs a) {
    pdl_wait();  // the kernel before this one in the stream has completed
    pdl_launch_dependents();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int b = blockIdx.x, tid = threadIdx.x;
    const StepDims sd = clamp_step(a.steps[b], a.n_levels, a.n_slots, a.max_tt, a.max_k, a.vocab);
    const int k = sd.k, kk = k * k;
    const int d = (a.emit_level >= 0) ? min(sd.d, a.emit_level + 1) : sd.d;  // levels ranked by this launch
    const int n_cand = k + (d - 1) * kk;
    const int m = min(sd.tt - 1, n_cand);
    const int n = m + 1;

    double* score = reinterpret_cast<double*>(smem_raw);                  // [cand_cap]
    int* sorted = reinterpret_cast<int*>(score + a.cand_cap);             // [cand_cap] per level, by rank
    int* node_of = sorted + a.cand_cap;                                   // [cand_cap] level rank, then node index
    int* frontier = node_of + a.cand_cap;                                 // [max_depth][max_k]
    int* s_parent = frontier + RESPS_MAX_DEPTH * RESPS_MAX_K;             // [max_tt] node -> parent node
    int* s_flag = s_parent + RESPS_MAX_TT;                                // [max_tt] has-child flags
    int* s_warp = s_flag + RESPS_MAX_TT;                                  // [33] scan scratch

    const int64_t row0 = static_cast<int64_t>(b) * a.max_rows;
    auto cand_level = [&](int c) { return (c < k) ? 0 : 1 + (c - k) / kk; };
    auto cand_row = [&](int c) {  // scanned row the candidate's token comes from
        if (c < k) return 0;
        const int j = 1 + (c - k) / kk, i = (c - k) % kk;
        return 1 + (j - 1) * k + i / k;
    };
    auto cand_rank_in_row = [&](int c) { return (c < k) ? c : ((c - k) % kk) % k; };
    auto cand_parent = [&](int c) {  // candidate index of the parent, -1 for the root
        if (c < k) return -1;
        const int j = 1 + (c - k) / kk, i = (c - k) % kk;
        return frontier[(j - 1) * RESPS_MAX_K + i / k];
    };

    // ---- every candidate's own log-probability, in one round trip to global memory (the rows
    // a level reads do not depend on the levels before it) -----------------------------------
    for (int c = tid; c < n_cand; c += kTreeThreads) {
        const int64_t row = row0 + cand_row(c);
        const double lp = static_cast<double>(a.row_val[row * a.max_k + cand_rank_in_row(c)]) - a.row_lse[row];
        score[c] = fmin(lp, 0.0);
    }
    // ---- level 0 ---------------------------------------------------------------
    if (tid < k) {
        sorted[tid] = tid;
        frontier[tid] = tid;
    }
    __syncthreads();

    // ---- levels 1..d-1 -----------------------------------------------------------
    for (int j = 1; j < d; ++j) {
        const int base = k + (j - 1) * kk;
        for (int i = tid; i < kk; i += kTreeThreads)
            score[base + i] += score[frontier[(j - 1) * RESPS_MAX_K + i / k]];
        __syncthreads();
        // rank inside the level by counting, eight threads per candidate (independent shared-memory
        // reads pipeline; a chain of dependent binary-search steps does not)
        for (int i0 = 0; i0 < kk; i0 += kTreeThreads / 8) {
            const int i = i0 + (tid >> 3), sub = tid & 7;
            const bool live = i < kk;
            const int c = base + (live ? i : 0);
            const double s = score[c];
            int rank = 0;
            if (live)
                for (int i2 = sub; i2 < kk; i2 += 8) rank += before(score[base + i2], base + i2, s, c) ? 1 : 0;
            rank += __shfl_xor_sync(kFull, rank, 1);
            rank += __shfl_xor_sync(kFull, rank, 2);
            rank += __shfl_xor_sync(kFull, rank, 4);
            if (live && sub == 0) {
                sorted[base + rank] = c;
                if (rank < k) frontier[j * RESPS_MAX_K + rank] = c;
            }
        }
        __syncthreads();
    }

    if (a.emit_level >= 0) {
        // ---- level form: the frontier after level j, for the draft model's next pass ------------------
        // Member p is draft node 1 + j k + p (the root is draft node 0, the frontier of level i occupies
        // 1 + i k .. i k + k): token, the slot of its parent in the previous frontier, position id, the
        // ancestor-or-self mask over draft nodes (only while they fit 128 bits) and its score.
        const int j = a.emit_level;
        if (j < sd.d && tid < k) {
            const int c = frontier[j * RESPS_MAX_K + tid];
            const int64_t of = static_cast<int64_t>(b) * a.max_k + tid;
            a.fr.tokens[of] = a.row_id[(row0 + cand_row(c)) * a.max_k + cand_rank_in_row(c)];
            a.fr.parent_slot[of] = (j == 0) ? -1 : ((c - (k + (j - 1) * kk)) / k);
            a.fr.position_ids[of] = sd.L + j + 1;
            a.fr.node_index[of] = 1 + j * k + tid;
            if (a.fr.score) a.fr.score[of] = score[c];
            unsigned long long lo = 1ull, hi = 0ull;  // the root
            if (1 + (j + 1) * k <= 128) {
                int cc = c, slot = tid;
                for (int jj = j; jj >= 0; --jj) {
                    const int node = 1 + jj * k + slot;
                    if (node < 64)
                        lo |= 1ull << node;
                    else
                        hi |= 1ull << (node - 64);
                    if (jj > 0) {
                        slot = (cc - (k + (jj - 1) * kk)) / k;
                        cc = frontier[(jj - 1) * RESPS_MAX_K + slot];
                    }
                }
            } else {
                lo = 0ull;
            }
            a.fr.mask[of * 2 + 0] = lo;
            a.fr.mask[of * 2 + 1] = hi;
        }
        // (a sequence whose own d is below j + 1 has nothing at this level: its entries stay untouched)
        if (tid == 0 && sd.clamped) atomicOr(a.status, RESPS_STATUS_STEP_CLAMPED);
        return;
    }

    // ---- global rerank: keep the m best of all candidates -------------------------
    for (int c = tid; c < n_cand; c += kTreeThreads) node_of[c] = 0;
    __syncthreads();
    // sorted[] holds, per level, the candidates by level rank; invert it to get each one's rank
    for (int i = tid; i < n_cand; i += kTreeThreads) {
        const int c = sorted[i];
        const int j = cand_level(c);
        const int lbase = (j == 0) ? 0 : k + (j - 1) * kk;
        const int lrank = i - lbase;
        int keep = 0;
        if (lrank < m) {
            int g = lrank;
            const double s = score[c];
            for (int q = 0; q < d && g < m; ++q) {
                if (q == j) continue;
                const int qbase = (q == 0) ? 0 : k + (q - 1) * kk;
                const int qn = (q == 0) ? k : kk;
                g += count_before(sorted + qbase, min(qn, m), score, s, c);
            }
            keep = (g < m);
        }
        node_of[c] = keep;
    }
    __syncthreads();

    // ---- node index = 1 + kept candidates with a lower index ------------------------
    const int per = (n_cand + kTreeThreads - 1) / kTreeThreads;
    const int c0 = min(tid * per, n_cand), c1 = min(c0 + per, n_cand);
    int cnt = 0;
    for (int c = c0; c < c1; ++c) cnt += node_of[c];
    int total;
    int run = block_exclusive_scan(cnt, s_warp, total);
    const int64_t ob = static_cast<int64_t>(b) * a.max_tt;
    for (int c = c0; c < c1; ++c) {
        if (node_of[c]) {
            node_of[c] = 1 + run++;
        } else {
            node_of[c] = 0;
        }
    }
    __syncthreads();
    // The draft row every node's children were taken from (kept in the workspace for the acceptance
    // under sampling, which needs the draft distribution behind every tried child): the root's is row
    // (0, 0); the p-th member of the frontier after level j < d-1 was given row (j+1, p).
    for (int i = tid; i < n; i += kTreeThreads) a.node_row[ob + i] = (i == 0) ? 0 : -1;
    __syncthreads();
    for (int e = tid; e < (d - 1) * k; e += kTreeThreads) {
        const int j = e / k, p = e - j * k;
        const int i = node_of[frontier[j * RESPS_MAX_K + p]];
        if (i > 0) a.node_row[ob + i] = (j + 1) * RESPS_MAX_K + p;
    }
    // `total` equals m by construction of the ranks.
    for (int c = tid; c < n_cand; c += kTreeThreads) {
        const int i = node_of[c];
        if (i == 0) continue;
        const int pc = cand_parent(c);
        const int pn = (pc < 0) ? 0 : node_of[pc];
        const int dep = cand_level(c) + 1;
        a.tokens[ob + i] = a.row_id[(row0 + cand_row(c)) * a.max_k + cand_rank_in_row(c)];
        a.parent[ob + i] = pn;
        a.depth[ob + i] = dep;
        a.position_ids[ob + i] = sd.L + dep;
        s_parent[i] = pn;
    }
    if (tid == 0) {
        a.tokens[ob] = a.root_token[b];
        a.parent[ob] = -1;
        a.depth[ob] = 0;
        a.position_ids[ob] = sd.L;
        s_parent[0] = -1;
        a.n_nodes[b] = n;
        if (sd.clamped || total != m) atomicOr(a.status, RESPS_STATUS_STEP_CLAMPED);
    }
    if (tid < RESPS_MAX_TT) s_flag[tid] = 0;
    __syncthreads();

    // ---- ancestor masks, leaves, retrieve rows --------------------------------------
    const int rs = a.max_depth + 1;
    if (tid < n) {
        unsigned long long lo = 0ull, hi = 0ull;
        int cur = tid, dep = 0;
        while (cur >= 0 && dep <= RESPS_MAX_DEPTH) {
            if (cur < 64)
                lo |= 1ull << cur;
            else
                hi |= 1ull << (cur - 64);
            cur = s_parent[cur];
            ++dep;
        }
        a.mask[(ob + tid) * 2 + 0] = lo;
        a.mask[(ob + tid) * 2 + 1] = hi;
        if (tid > 0) s_flag[s_parent[tid]] = 1;
    }
    __syncthreads();
    if (tid < RESPS_MAX_TT) {  // 4 warps: rank the leaves with ballots
        const bool leaf = (tid < n) && !s_flag[tid];
        const unsigned bal = __ballot_sync(kFull, leaf);
        if ((tid & 31) == 0) s_warp[tid >> 5] = __popc(bal);
        // named barrier over the first 128 threads only
        asm volatile("bar.sync 1, 128;");
        int row = __popc(bal & ((1u << (tid & 31)) - 1u));
        for (int w = 0; w < (tid >> 5); ++w) row += s_warp[w];
        if (leaf) {
            int32_t* out = a.retrieve + (ob + row) * rs;
            int len = 0;
            for (int cur = tid; cur >= 0 && len < rs; cur = s_parent[cur]) ++len;
            for (int t = len; t < rs; ++t) out[t] = -1;
            int cur = tid;
            for (int t = len - 1; t >= 0; --t) {
                out[t] = cur;
                cur = s_parent[cur];
            }
        }
        if (tid == 0) a.n_leaves[b] = s_warp[0] + s_warp[1] + s_warp[2] + s_warp[3];
    }
}

}  // namespace

static size_t tree_smem_bytes(int cand_cap) {
    return static_cast<size_t>(cand_cap) * (sizeof(double) + 2 * sizeof(int)) +
           sizeof(int) * (RESPS_MAX_DEPTH * RESPS_MAX_K + 2 * RESPS_MAX_TT + 40);
}

cudaError_t launch_tree_build(const resps_ctx* ctx, const resps_step* d_steps, int batch,
                              int n_levels, int n_slots, const int32_t* root_token,
                              int32_t* tokens, int32_t* parent, int32_t* depth, int32_t* position_ids,
                              uint64_t* mask, int32_t* retrieve, int32_t* n_leaves, int32_t* n_nodes,
                              cudaStream_t st) {
    const resps_shape& s = ctx->shape;
    TreeArgs a;
    a.steps = d_steps;
    a.n_levels = n_levels, a.n_slots = n_slots;
    a.vocab = s.vocab, a.max_tt = s.max_tt, a.max_k = s.max_k, a.max_depth = s.max_depth;
    a.max_rows = ctx->ws.max_rows;
    a.row_val = ctx->ws.row_val, a.row_id = ctx->ws.row_id, a.row_lse = ctx->ws.row_lse;
    a.root_token = root_token;
    a.tokens = tokens, a.parent = parent, a.depth = depth, a.position_ids = position_ids;
    a.mask = mask, a.retrieve = retrieve, a.n_leaves = n_leaves, a.n_nodes = n_nodes;
    a.node_row = ctx->ws.node_row;
    a.status = ctx->ws.status;
    a.cand_cap = s.max_k + (s.max_depth - 1) * s.max_k * s.max_k;
    a.emit_level = -1;
    a.fr = FrontierOut{};
    const size_t smem = tree_smem_bytes(a.cand_cap);
    return launch_pdl(tree_build_kernel, dim3(batch), dim3(kTreeThreads), smem, st, a);
}

cudaError_t launch_tree_level(const resps_ctx* ctx, const resps_step* d_steps, int batch, int n_levels, int n_slots,
                              int level, const FrontierOut& out, cudaStream_t st) {
    const resps_shape& s = ctx->shape;
    TreeArgs a = {};
    a.steps = d_steps;
    a.n_levels = n_levels, a.n_slots = n_slots;
    a.vocab = s.vocab, a.max_tt = s.max_tt, a.max_k = s.max_k, a.max_depth = s.max_depth;
    a.max_rows = ctx->ws.max_rows;
    a.row_val = ctx->ws.row_val, a.row_id = ctx->ws.row_id, a.row_lse = ctx->ws.row_lse;
    a.node_row = ctx->ws.node_row;
    a.status = ctx->ws.status;
    a.cand_cap = s.max_k + (s.max_depth - 1) * s.max_k * s.max_k;
    a.emit_level = level;
    a.fr = out;
    return launch_pdl(tree_build_kernel, dim3(batch), dim3(kTreeThreads), tree_smem_bytes(a.cand_cap), st, a);
}

// Largest k + (d-1)k^2 the shared-memory arrays can hold.
int tree_candidate_limit() { return (200 * 1024 - 4096) / static_cast<int>(sizeof(double) + 2 * sizeof(int)); }

cudaError_t tree_setup(resps_ctx*) {
    return cudaFuncSetAttribute(tree_build_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                200 * 1024);
}

}  // namespace resps
