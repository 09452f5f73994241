// Draft-tree build from the scanned rows (Section 3.2, "Draft Tree Expansion":
// cumulative score V_i along the root path, the k best of a layer are expanded;
// "Confidence-Based Candidate Reranking": all expanded tokens are reranked and the
// best TT-1 kept; Algorithm 2, tree-building loop).  One CTA per sequence; integer
// and fp64 work on at most k + (d-1)k^2 candidates, all in shared memory.
//
// Every level's candidates are k lists (one per frontier member), each already in the method's
// order because a scanned row is sorted; a candidate's rank inside its level is its place in its own
// list plus, for every other list, a binary search (one thread per candidate and list).  Its rank in
// the global rerank is its level rank plus binary searches over the other levels' sorted heads, and
// only the first TT-1 of a level can be kept at all.
#include <cmath>

#include "common.cuh"

namespace resps {
namespace {

constexpr int kTreeThreads = 1024;
constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kStride = 8;                       // rerank: level ranks between two coarse probes
constexpr int kProbes = RESPS_MAX_TT / kStride;  // coarse probes per level
constexpr int kTokPrefetch = 2;  // token ids of the first 2 x 1024 candidates travel in registers
static_assert(kTreeThreads == 1024, "the node-index scan assumes 32 warps");

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
    int setup_before_wait;  // 1: a scan or merge kernel of the same call runs directly before this kernel
};

// Path scores are compared as integers: the map below keeps the order of finite doubles (and their
// equality, zero being stored as +0); an integer key turns "at least" into "above key - 1", which
// spares the searches the tie-break read.  The map is its own inverse.
__device__ __forceinline__ long long score_key(double s) {
    const long long bits = __double_as_longlong(s + 0.0);
    return bits ^ ((bits >> 63) & 0x7FFFFFFFFFFFFFFFll);
}
__device__ __forceinline__ double key_score(long long key) {
    return __longlong_as_double(key ^ ((key >> 63) & 0x7FFFFFFFFFFFFFFFll));
}

// Exact floor(e / d) for 0 <= e < 2^22 and 1 <= d <= 2^10: the quotient's fraction is at least
// 0.5 / d away from an integer after the half is added, far more than the float rounding.
struct FastDiv {
    float inv;
    __device__ explicit FastDiv(int d) : inv(1.0f / static_cast<float>(d)) {}
    __device__ __forceinline__ int div(int e) const { return __float2int_rd((static_cast<float>(e) + 0.5f) * inv); }
};

// Leading entries of the descending key list `keys[0..n)` that are above `thr`; `top` is the largest
// power of two <= n (0 for an empty list).  A fixed number of steps without data-dependent branches.
//
// Candidate order of the method: larger score first, equal scores by lower candidate index.  Two
// candidates of different lists of a level, or of different levels, compare by index the same way
// for the whole list, so "before (key, c)" is "key above thr" with thr = key - 1 where the list's
// indices are the lower ones and thr = key otherwise.
__device__ __forceinline__ int count_above(const long long* keys, int n, int top, long long thr) {
    int pos = 0;
    for (int half = top; half > 0; half >>= 1) {
        const int t = pos + half;
        if (t <= n && keys[t - 1] > thr) pos = t;
    }
    return pos;
}
__device__ __forceinline__ int pow2_floor(int n) { return (n > 0) ? (1 << (31 - __clz(n))) : 0; }

__global__ void __launch_bounds__(kTreeThreads, 1) tree_build_kernel(const TreeArgs a) {
    // The step parameters were written at least two kernels ago (a scan or a merge kernel of the same
    // call always sits between their writer and this kernel, and every kernel of the library signals its
    // dependents only after its own wait), so they are read, and everything that follows from them is
    // set up, before the wait for the rows: under the tail of the kernel that scans them.  (Where no such
    // kernel precedes this one -- the last call of the level form -- the wait comes first.)
    if (!a.setup_before_wait) pdl_wait();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int b = blockIdx.x, tid = threadIdx.x;
    const StepDims sd = clamp_step(a.steps[b], a.n_levels, a.n_slots, a.max_tt, a.max_k, a.vocab);
    const int k = sd.k, kk = k * k;
    const int d = (a.emit_level >= 0) ? min(sd.d, a.emit_level + 1) : sd.d;  // levels ranked by this launch
    const int n_cand = k + (d - 1) * kk;
    const int m = min(sd.tt - 1, n_cand);
    const int n = m + 1;

    long long* skey = reinterpret_cast<long long*>(smem_raw);             // [cand_cap] own log-prob (as a double), then the key of the path score
    long long* head_key = skey + a.cand_cap;                              // [max_depth][max_tt] keys of a level's first ranks
    double* fscore = reinterpret_cast<double*>(head_key + RESPS_MAX_DEPTH * RESPS_MAX_TT);  // [max_depth][max_k] frontier scores
    int* node_of = reinterpret_cast<int*>(fscore + RESPS_MAX_DEPTH * RESPS_MAX_K);  // [cand_cap] rank counters, level rank, then node index
    int* frontier = node_of + a.cand_cap;                                 // [max_depth][max_k]
    int* s_parent = frontier + RESPS_MAX_DEPTH * RESPS_MAX_K;             // [max_tt] node -> parent node
    int* s_flag = s_parent + RESPS_MAX_TT;                                // [max_tt] has-child flags
    int* s_warp = s_flag + RESPS_MAX_TT;                                  // [2][32] scan scratch
    int* probe = s_warp + 64;                                             // [max_depth][kProbes] rerank counters, coarse
    int* fine = probe + RESPS_MAX_DEPTH * kProbes;                        // [max_depth][kStride] rerank counters, fine
    int* n_coarse = fine + RESPS_MAX_DEPTH * kStride;                     // [max_depth] probes kept
    int* n_fine = n_coarse + RESPS_MAX_DEPTH;                             // [max_depth] kept after the last kept probe

    // The kernel is bound by instruction issue (one CTA of 32 warps), so index arithmetic by the
    // run-time k, k^2 and d goes through an exact float reciprocal (operands stay below 2^22).
    const FastDiv by_k(k), by_kk(kk), by_d(d);
    const int64_t row0 = static_cast<int64_t>(b) * a.max_rows;
    struct Cand {
        int level, list, place;  // level, list inside the level (frontier slot of the parent), place in the list
    };
    auto decode = [&](int c) {
        Cand r;
        if (c < k) {
            r.level = 0, r.list = 0, r.place = c;
        } else {
            const int t = c - k, jm1 = by_kk.div(t), i = t - jm1 * kk;
            r.level = jm1 + 1;
            r.list = by_k.div(i);
            r.place = i - r.list * k;
        }
        return r;
    };
    auto cand_row = [&](const Cand& r) { return (r.level == 0) ? 0 : 1 + (r.level - 1) * k + r.list; };

    // ---- every candidate's own log-probability, in one round trip to global memory (the rows
    // a level reads do not depend on the levels before it); the token ids of the first candidates
    // come along in registers for the outputs at the end ---------------------------------------
    const Cand own = decode(min(tid, n_cand - 1));  // candidate tid, reused by the later passes over candidates
    int tok_pre[kTokPrefetch];
#pragma unroll
    for (int i = 0; i < kTokPrefetch; ++i) tok_pre[i] = 0;
    for (int i = tid; i < RESPS_MAX_DEPTH * (kProbes + kStride + 2); i += kTreeThreads) probe[i] = 0;
    // the first pass of the per-level loops below has the same index arithmetic at every level
    const int pair_i = by_k.div(tid), pair_p2 = tid - pair_i * k, pair_p = by_k.div(pair_i);  // pair tid = (candidate, list)
    const int k_top = pow2_floor(k);
    if (a.setup_before_wait) pdl_wait();  // the kernel before this one in the stream has completed: the scanned rows are there
    pdl_launch_dependents();
    for (int c = tid, i = 0; c < n_cand; c += kTreeThreads, ++i) {
        const Cand r = (i == 0) ? own : decode(c);
        const int64_t row = row0 + cand_row(r);
        const int64_t at = row * a.max_k + r.place;
        if (i < kTokPrefetch && a.emit_level < 0) {
#pragma unroll
            for (int u = 0; u < kTokPrefetch; ++u)
                if (u == i) tok_pre[u] = a.row_id[at];
        }
        // (+ 0.0 stores a zero as +0, so that equal scores have equal keys)
        const double lp = fmin(static_cast<double>(a.row_val[at]) - a.row_lse[row], 0.0) + 0.0;
        skey[c] = (c < k) ? score_key(lp) : __double_as_longlong(lp);
        node_of[c] = (c < k) ? c : 0;  // level 0 is ranked as scanned; the other levels count from 0
    }
    __syncthreads();
    // ---- level 0 ---------------------------------------------------------------
    if (tid < k) {
        frontier[tid] = tid;
        fscore[tid] = key_score(skey[tid]);
        head_key[tid] = skey[tid];
    }
    __syncthreads();

    // ---- levels 1..d-1 -----------------------------------------------------------
    for (int j = 1; j < d; ++j) {
        const int base = k + (j - 1) * kk;
        const double* fs = fscore + (j - 1) * RESPS_MAX_K;
        // path score = own log-probability + the parent's path score, kept as its key
        for (int i = tid; i < kk; i += kTreeThreads) {
            const int p = (i == tid) ? pair_i : by_k.div(i);  // (pair_i = tid / k)
            skey[base + i] = score_key(__longlong_as_double(skey[base + i]) + fs[p]);
        }
        __syncthreads();
        // one thread per (candidate, other list): candidates of that list ranking before it
        for (int e = tid; e < kk * k; e += kTreeThreads) {
            int i = pair_i, p2 = pair_p2, p = pair_p;
            if (e != tid) {
                i = by_k.div(e), p2 = e - i * k;
                p = by_k.div(i);
            }
            if (p2 == p) continue;
            const int c = base + i;
            const int cnt = count_above(skey + base + p2 * k, k, k_top, skey[c] - ((p2 < p) ? 1 : 0));
            if (cnt) atomicAdd(&node_of[c], cnt);
        }
        __syncthreads();
        // level rank = place in the own list + the counts; the k best form the next frontier
        for (int i = tid; i < kk; i += kTreeThreads) {
            const int c = base + i, p = (i == tid) ? pair_i : by_k.div(i);
            const int rank = (i - p * k) + node_of[c];
            const long long key = skey[c];
            node_of[c] = rank;
            if (rank < k) {
                frontier[j * RESPS_MAX_K + rank] = c;
                fscore[j * RESPS_MAX_K + rank] = key_score(key);
            }
            if (rank < RESPS_MAX_TT) head_key[j * RESPS_MAX_TT + rank] = key;
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
            const Cand r = decode(c);
            a.fr.tokens[of] = a.row_id[(row0 + cand_row(r)) * a.max_k + r.place];
            a.fr.parent_slot[of] = (j == 0) ? -1 : ((c - (k + (j - 1) * kk)) / k);
            a.fr.position_ids[of] = sd.L + j + 1;
            a.fr.node_index[of] = 1 + j * k + tid;
            if (a.fr.score) a.fr.score[of] = key_score(skey[c]);
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
    // Inside a level the global rank grows with the level rank, so a level keeps a prefix of its
    // sorted order and only the prefix length is needed.  A candidate's global rank is its level
    // rank plus, per other level, a binary search over that level's first m scores (one thread per
    // candidate and level).  Coarse pass: every kStride-th level rank; fine pass: the kStride-1
    // ranks after the last probe that was kept.
    const int mm = min(kk, m), m0 = min(k, m);
    auto level_head = [&](int j) { return (j == 0) ? m0 : mm; };
    const int mm_top = pow2_floor(mm), m0_top = pow2_floor(m0);
    auto others_before = [&](int j, int i, int q) {  // of level q's first m, those before (level j, rank i)
        const long long key = head_key[j * RESPS_MAX_TT + i];
        return count_above(head_key + q * RESPS_MAX_TT, level_head(q), (q == 0) ? m0_top : mm_top, key - ((q < j) ? 1 : 0));
    };
    const int n_probe = (mm + kStride - 1) / kStride;
    const FastDiv by_probe(max(n_probe, 1)), by_fine(kStride - 1);
    for (int e = tid; e < d * n_probe * d; e += kTreeThreads) {
        const int slot = by_d.div(e), q = e - slot * d;
        const int j = by_probe.div(slot), u = slot - j * n_probe;
        if (q == j || u * kStride >= level_head(j)) continue;
        const int cnt = others_before(j, u * kStride, q);
        if (cnt) atomicAdd(&probe[j * kProbes + u], cnt);
    }
    __syncthreads();
    for (int e = tid; e < d * n_probe; e += kTreeThreads) {
        const int j = by_probe.div(e), u = e - j * n_probe;
        if (u * kStride < level_head(j) && u * kStride + probe[j * kProbes + u] < m) atomicAdd(&n_coarse[j], 1);
    }
    __syncthreads();
    for (int e = tid; e < d * (kStride - 1) * d; e += kTreeThreads) {
        const int slot = by_d.div(e), q = e - slot * d;
        const int j = by_fine.div(slot), w = slot - j * (kStride - 1) + 1;
        const int kept = n_coarse[j];
        const int i = (kept - 1) * kStride + w;
        if (q == j || kept == 0 || i >= level_head(j)) continue;
        const int cnt = others_before(j, i, q);
        if (cnt) atomicAdd(&fine[j * kStride + w], cnt);
    }
    __syncthreads();
    for (int e = tid; e < d * (kStride - 1); e += kTreeThreads) {
        const int j = by_fine.div(e), w = e - j * (kStride - 1) + 1;
        const int kept = n_coarse[j];
        const int i = (kept - 1) * kStride + w;
        if (kept > 0 && i < level_head(j) && i + fine[j * kStride + w] < m) atomicAdd(&n_fine[j], 1);
    }
    __syncthreads();
    // level j keeps its first keep_of(j) ranks
    auto keep_of = [&](int j) { return (n_coarse[j] > 0) ? (n_coarse[j] - 1) * kStride + 1 + n_fine[j] : 0; };

    // ---- node index = 1 + kept candidates with a lower index ------------------------
    const int lane = tid & 31, warp = tid >> 5;
    int total = 0;
    for (int c0 = 0, it = 0; c0 < n_cand; c0 += kTreeThreads, ++it) {
        const int c = c0 + tid;
        const int level = (it == 0) ? own.level : decode(min(c, n_cand - 1)).level;
        const bool keep = (c < n_cand) && (node_of[c] < keep_of(level));
        const unsigned bal = __ballot_sync(kFull, keep);
        int* sw = s_warp + (it & 1) * 32;
        if (lane == 0) sw[warp] = __popc(bal);
        __syncthreads();
        int inc = sw[lane];  // kTreeThreads / 32 == 32 warps
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(kFull, inc, o);
            if (lane >= o) inc += t;
        }
        const int before_warp = __shfl_sync(kFull, inc, warp) - __popc(bal);
        const int chunk_total = __shfl_sync(kFull, inc, 31);
        if (c < n_cand) node_of[c] = keep ? 1 + total + before_warp + __popc(bal & ((1u << lane) - 1u)) : 0;
        total += chunk_total;
    }
    const int64_t ob = static_cast<int64_t>(b) * a.max_tt;
    __syncthreads();
    // The draft row every node's children were taken from (kept in the workspace for the acceptance
    // under sampling, which needs the draft distribution behind every tried child): the root's is row
    // (0, 0); the p-th member of the frontier after level j < d-1 was given row (j+1, p).
    for (int i = tid; i < n; i += kTreeThreads) a.node_row[ob + i] = (i == 0) ? 0 : -1;
    __syncthreads();
    for (int e = tid; e < (d - 1) * k; e += kTreeThreads) {
        const int j = by_k.div(e), p = e - j * k;
        const int i = node_of[frontier[j * RESPS_MAX_K + p]];
        if (i > 0) a.node_row[ob + i] = (j + 1) * RESPS_MAX_K + p;
    }
    // `total` equals m by construction of the ranks.
    for (int c = tid, it = 0; c < n_cand; c += kTreeThreads, ++it) {
        const int i = node_of[c];
        if (i == 0) continue;
        const Cand r = (it == 0) ? own : decode(c);
        const int pn = (r.level == 0) ? 0 : node_of[frontier[(r.level - 1) * RESPS_MAX_K + r.list]];
        const int dep = r.level + 1;
        int tok = 0;
        if (it < kTokPrefetch) {
#pragma unroll
            for (int u = 0; u < kTokPrefetch; ++u)
                if (u == it) tok = tok_pre[u];
        } else {
            tok = a.row_id[(row0 + cand_row(r)) * a.max_k + r.place];
        }
        a.tokens[ob + i] = tok;
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

constexpr size_t kTreeFixedSmem = sizeof(double) * (RESPS_MAX_DEPTH * RESPS_MAX_TT + RESPS_MAX_DEPTH * RESPS_MAX_K) +
                                  sizeof(int) * (RESPS_MAX_DEPTH * RESPS_MAX_K + 2 * RESPS_MAX_TT + 64 +
                                                 RESPS_MAX_DEPTH * (kProbes + kStride + 2));
constexpr size_t kTreeSmemCap = 200 * 1024;

static size_t tree_smem_bytes(int cand_cap) {
    return static_cast<size_t>(cand_cap) * (sizeof(double) + sizeof(int)) + kTreeFixedSmem;
}

cudaError_t launch_tree_build(const resps_ctx* ctx, const resps_step* d_steps, int batch,
                              int n_levels, int n_slots, const int32_t* root_token,
                              int32_t* tokens, int32_t* parent, int32_t* depth, int32_t* position_ids,
                              uint64_t* mask, int32_t* retrieve, int32_t* n_leaves, int32_t* n_nodes,
                              cudaStream_t st, bool after_scan) {
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
    a.setup_before_wait = after_scan ? 1 : 0;
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
    a.setup_before_wait = 1;  // the scan of this level's rows runs directly before
    a.fr = out;
    return launch_pdl(tree_build_kernel, dim3(batch), dim3(kTreeThreads), tree_smem_bytes(a.cand_cap), st, a);
}

// Largest k + (d-1)k^2 the shared-memory arrays can hold.
int tree_candidate_limit() {
    return static_cast<int>((kTreeSmemCap - kTreeFixedSmem) / (sizeof(double) + sizeof(int)));
}

cudaError_t tree_setup(resps_ctx*) {
    return cudaFuncSetAttribute(tree_build_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                static_cast<int>(kTreeSmemCap));
}

}  // namespace resps
