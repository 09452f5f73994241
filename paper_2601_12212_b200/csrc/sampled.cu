// Verification and acceptance under sampling, temperature T > 0 (Section 3.2, "Acceptance
// Criterion": a draft token y is accepted with probability min(1, P_T(y) / P_d(y)); Section 4.1,
// "Lossless Output Fidelity": rejection-based correction keeps the target's distribution).
//
// For a chain of draft tokens this is the paper's rule with the correction step of the
// speculative-sampling papers it cites (on the first rejection the token is drawn from the
// normalised residual max(0, P_T - P_d); after a chain accepted in full, from P_T).  In a tree the
// children of the current node are tried in node order; after a rejected child x the target side
// becomes the normalised residual max(0, p - q), the draft side q without x, renormalised, and the
// next sibling is tried against those; when no child is left the token is drawn from the residual.
//
// All of it is a walk of at most max_depth + 1 nodes, but each step of the walk needs sums over the
// whole vocabulary (normalisers of softmax and of residuals, the cumulative sum the token is drawn
// from).  A thread-block cluster of 8 CTAs serves one sequence: every CTA takes an eighth of the
// vocabulary, every CTA writes its partial sums into every peer's shared memory behind the hardware
// cluster barrier (no spinning anywhere), and every CTA then takes the same decision from the same
// numbers.  Arithmetic is fp64 throughout: a decision (accept or not, which token) is a comparison of
// sums over 10^5 terms, and only at fp64 is the order of summation immaterial to it.
//
// The exponentials dominate, so each is taken once per visited node.  The target-side value P of
// every token of the CTA's slice lives in shared memory (in an L2-resident scratch when the slice is
// too large) and is brought up to date in place by the pass that needs it next -- first the division
// by the softmax sum, then one rejection round per pass.  The draft side is the raw exponentials Q in
// the scratch times one scalar (softmax sum and renormalisations are the same factor for every
// token; a removed token's entry is set to zero), so a pass reads 8 bytes per token from L2 and
// multiplies.  Only the thread that owns a token touches its values; (P, Q) of the current node's
// children, which every CTA needs for the decisions, are copied by their owners into a small table
// behind the same barrier that carries the sums (two tables in turn, so that a pass never writes the
// one being read).
#include <cmath>

#include "common.cuh"

namespace resps {
namespace {

constexpr int kClu = 8;             // CTAs per sequence
constexpr int kSampThreads = 1024;
constexpr unsigned kFull = 0xFFFFFFFFu;

struct SampledArgs {
    const resps_step* steps;
    const int32_t* n_nodes;
    const float* target;
    int64_t ld_b, ld_row;
    const float* draft;
    int64_t dld_b, dld_level, dld_row;
    const int32_t* node_row;  // [batch][max_tt]: level * RESPS_MAX_K + slot of the row a node's children came from
    double inv_t;             // 1 / temperature
    double temperature;
    const int32_t *tokens, *parent;
    const double *u_accept, *u_sample;
    int vocab, max_tt, max_depth, max_k;
    int32_t *accept_path, *accept_len, *out_tokens;
    resps_step* steps_next;
    double* scratch;  // [batch][kScratchPerSeq] small words, then [batch][kClu][2][per_thr * kSampThreads] (P, Q)
    int64_t state_per_cta;  // doubles of one CTA's p (or q) array
    int staged;             // 1: a row's slice fits the staging area in shared memory
    int p_in_smem;          // 1: the target-side values live in shared memory (else in the scratch)
};
constexpr int kTableAt = 4 * kClu + 8;
constexpr int kScratchPerSeq = kTableAt + 2 * 2 * RESPS_MAX_K;  // two alternating sets of pairs of partials, the
                                                                // drawn token, two alternating tables of the children's (p, q)

__device__ __forceinline__ unsigned cluster_rank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

struct Pair {
    double x, y;
};

// Two sums (or two maxima) over the CTA at once, result in every thread.
template <bool MAX>
__device__ __forceinline__ Pair block_reduce2(Pair v, double* s_red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double wx = __shfl_xor_sync(kFull, v.x, o), wy = __shfl_xor_sync(kFull, v.y, o);
        v.x = MAX ? fmax(v.x, wx) : v.x + wx;
        v.y = MAX ? fmax(v.y, wy) : v.y + wy;
    }
    __syncthreads();  // s_red is free again
    if (lane == 0) s_red[2 * warp] = v.x, s_red[2 * warp + 1] = v.y;
    __syncthreads();
    Pair r = {s_red[0], s_red[1]};
    for (int w = 1; w < kSampThreads / 32; ++w) {
        r.x = MAX ? fmax(r.x, s_red[2 * w]) : r.x + s_red[2 * w];
        r.y = MAX ? fmax(r.y, s_red[2 * w + 1]) : r.y + s_red[2 * w + 1];
    }
    return r;
}

// Store one double into the shared memory of CTA `peer` of the cluster, at the address `local` has here.
__device__ __forceinline__ void store_to_peer(double* local, unsigned peer, double v) {
    const uint32_t mine = static_cast<uint32_t>(__cvta_generic_to_shared(local));
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(mine), "r"(peer));
    asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(remote), "d"(v) : "memory");
}

// The same over the cluster: every CTA writes its result into every peer's shared memory (slot
// `rank` of `s_peer[set]`), the hardware cluster barrier orders the writes, and every thread adds the
// eight up in rank order, so all CTAs hold the same bits.  `set` alternates between consecutive
// reductions (a set is written again only after everyone has read it: the barrier of the reduction
// in between).  The barrier also makes the children's table a pass has written visible to the cluster.
template <bool MAX>
__device__ __forceinline__ Pair cluster_reduce2(Pair v, double* s_red, double (*s_peer)[kClu][2], int& set, unsigned rank) {
    const Pair mine = block_reduce2<MAX>(v, s_red);
    if (threadIdx.x < kClu) {
        store_to_peer(&s_peer[set][rank][0], threadIdx.x, mine.x);
        store_to_peer(&s_peer[set][rank][1], threadIdx.x, mine.y);
    }
    cluster_barrier();
    Pair r = {s_peer[set][0][0], s_peer[set][0][1]};
    for (int c = 1; c < kClu; ++c) {
        r.x = MAX ? fmax(r.x, s_peer[set][c][0]) : r.x + s_peer[set][c][0];
        r.y = MAX ? fmax(r.y, s_peer[set][c][1]) : r.y + s_peer[set][c][1];
    }
    set ^= 1;
    return r;
}

// What the stored target-side value of a token still lacks: the division by the softmax sum, or one
// rejection round (Section 3.2, "Acceptance Criterion": target side -> normalised max(0, p - q)).  The
// draft side is kept as the raw exponentials times one scalar for the whole row (the softmax sum and
// the renormalisations after every removal are the same factor for every token), with the entry of
// a removed token set to zero.
struct Pending {
    int kind;      // 0 nothing, 1 softmax sum, 2 a rejection round
    double a;      // reciprocal of the target's sum (kind 1) / of the residual's normaliser (kind 2; 0: residual empty, p is kept)
    double sq_old; // kind 2: the draft side's scalar as it was when the round's child was tried
    int x;         // kind 2: the rejected token
};
// A division by a normaliser is a multiplication by its fp64 reciprocal (one rounding more than the
// quotient; the decisions compare sums of 10^5 such terms and are taken with a margin far above that).
__device__ __forceinline__ double recip_or_zero(double s) { return s > 0.0 ? 1.0 / s : 0.0; }
__device__ __forceinline__ double apply(const Pending& pd, double p, double q_raw) {
    if (pd.kind == 1) return p * pd.a;
    if (pd.kind == 2 && pd.a > 0.0) return fmax(p - q_raw * pd.sq_old, 0.0) * pd.a;
    return p;
}

__global__ void __launch_bounds__(kSampThreads, 1) accept_sampled_kernel(const SampledArgs a) {
    pdl_wait();  // the kernel before this one in the stream has completed
    pdl_launch_dependents();
    __shared__ double s_red[2 * (kSampThreads / 32)];
    __shared__ double s_scan[kSampThreads / 32];
    __shared__ double s_peer[2][kClu][2];  // the cluster's partial results, written by the peers
    __shared__ int s_tok[RESPS_MAX_TT], s_par[RESPS_MAX_TT];
    __shared__ int s_children[RESPS_MAX_TT];
    __shared__ int s_decision;                  // accepted child, or -1
    __shared__ int s_nchild;
    const unsigned rank = cluster_rank();
    const int b = blockIdx.x / kClu, tid = threadIdx.x;
    const int n = min(max(a.n_nodes[b], 1), a.max_tt);
    const int64_t ob = static_cast<int64_t>(b) * a.max_tt;
    const int cap = a.max_depth + 1;
    double* scratch = a.scratch + static_cast<int64_t>(b) * kScratchPerSeq;
    int set = 0;
    if (tid < n) s_tok[tid] = a.tokens[ob + tid], s_par[tid] = a.parent[ob + tid];
    if (rank == 0 && tid < cap) {
        a.accept_path[b * cap + tid] = (tid == 0) ? 0 : -1;
        a.out_tokens[b * cap + tid] = -1;
    }
    __syncthreads();
    // this CTA's share of the vocabulary, and inside it this thread's contiguous run
    const int V = a.vocab;
    const int per_cta = (V + kClu - 1) / kClu;
    const int c_lo = min(V, static_cast<int>(rank) * per_cta), c_hi = min(V, c_lo + per_cta);
    const int per_thr = (per_cta + kSampThreads - 1) / kSampThreads;
    const int t_lo = min(c_hi, c_lo + tid * per_thr), t_hi = min(c_hi, t_lo + per_thr);
    // Target-side value P and raw draft-side weight Q of the token at place i of thread t's run: element
    // i * threads + t of the owning CTA's arrays, so that a warp's accesses of one pass are contiguous.
    // Q lives in the L2-resident scratch; P in shared memory when the slice fits, else in the scratch too.
    extern __shared__ __align__(16) unsigned char s_dyn[];
    double* state0 = a.scratch + static_cast<int64_t>(gridDim.x / kClu) * kScratchPerSeq +
                     (static_cast<int64_t>(b) * kClu + rank) * 2 * a.state_per_cta;
    double* P = a.p_in_smem ? reinterpret_cast<double*>(s_dyn) : state0;
    double* Q = state0 + a.state_per_cta;
    float* s_stage = reinterpret_cast<float*>(s_dyn + (a.p_in_smem ? sizeof(double) * a.state_per_cta : 0));  // [threads][per_thr + 1]
    double* table = scratch + kTableAt;  // [2][RESPS_MAX_K][2]
    // After a pass (and a CTA barrier): the owners copy (P, Q) of the children's tokens into table `par`.
    auto publish_children = [&](int par, int n_child) {
        __syncthreads();
        if (tid < n_child && tid < RESPS_MAX_K) {
            const int x = s_tok[s_children[tid]];
            if (x >= c_lo && x < c_hi) {
                const int in_cta = x - c_lo, t = in_cta / per_thr, i = in_cta - t * per_thr;
                double* dst = table + (par * RESPS_MAX_K + tid) * 2;
                __stcg(dst, P[static_cast<int64_t>(i) * kSampThreads + t]);
                __stcg(dst + 1, __ldcg(Q + static_cast<int64_t>(i) * kSampThreads + t));
            }
        }
    };
    // The CTA's slice of a row through the staging area: coalesced loads (consecutive threads, consecutive
    // tokens), token e of the slice parked at [e / per_thr][e % per_thr] with a padded row, from where
    // every thread reads its own run without bank conflicts.  Returns the maximum this thread saw.
    auto stage_row = [&](const float* row, bool store) {
        constexpr int kGroup = 8;  // loads in flight per thread
        const int n_cta = c_hi - c_lo;
        float fm = -INFINITY;
        for (int e0 = tid; e0 < n_cta; e0 += kGroup * kSampThreads) {
            float x[kGroup];
#pragma unroll
            for (int u = 0; u < kGroup; ++u) {
                const int e = e0 + u * kSampThreads;
                x[u] = (e < n_cta) ? __ldg(row + c_lo + e) : -INFINITY;
            }
#pragma unroll
            for (int u = 0; u < kGroup; ++u) {
                const int e = e0 + u * kSampThreads;
                if (e >= n_cta) break;
                if (store) {
                    const int t = e / per_thr, i = e - t * per_thr;
                    s_stage[t * (per_thr + 1) + i] = x[u];
                }
                fm = fmaxf(fm, x[u]);
            }
        }
        return fm;
    };

    int cur = 0, acc = 0;
    for (;;) {
        const float* trow = a.target + b * a.ld_b + cur * a.ld_row;
        // ---- the children of the current node, in node order --------------------------------------
        if (tid == 0) {
            int m = 0;
            if (acc < a.max_depth)  // (the path array holds max_depth + 1 nodes; a tree is never deeper)
                for (int c = 1; c < n; ++c)
                    if (s_par[c] == cur) s_children[m++] = c;
            s_nchild = m;
        }
        __syncthreads();  // (also: the previous node's readers are done with the staging area)
        const int n_child = s_nchild;
        const float* drow = nullptr;
        if (n_child > 0) {
            const int row = a.node_row[ob + cur];  // >= 0 for a node with children
            drow = a.draft + b * a.dld_b + (row / RESPS_MAX_K) * a.dld_level + (row % RESPS_MAX_K) * a.dld_row;
        }
        // ---- P_T(. | cur) = softmax(row / T) and the draft's P_d: maxima, then the exponentials (stored)
        // and their sums.  The staging area holds one row at a time: the target's while the maxima are
        // taken (the draft row is only looked at), then the draft's (read again, from L2) -------------
        float fm_t = -INFINITY, fm_d = -INFINITY;
        if (a.staged) {
            fm_t = stage_row(trow, true);
            if (drow) fm_d = stage_row(drow, false);
        } else {
            for (int v = t_lo; v < t_hi; ++v) {
                fm_t = fmaxf(fm_t, __ldg(trow + v));
                if (drow) fm_d = fmaxf(fm_d, __ldg(drow + v));
            }
        }
        // (the reduction's barriers also order the staging area)
        const Pair mx = cluster_reduce2<true>(Pair{static_cast<double>(fm_t), static_cast<double>(fm_d)}, s_red, s_peer,
                                              set, rank);
        const double mx_t = mx.x * a.inv_t, mx_d = mx.y * a.inv_t;
        Pair sum = {0.0, 0.0};
        for (int v = t_lo, i = 0; v < t_hi; ++v, ++i) {
            const float xt = a.staged ? s_stage[tid * (per_thr + 1) + i] : __ldg(trow + v);
            const double wt = exp(static_cast<double>(xt) * a.inv_t - mx_t);
            P[static_cast<int64_t>(i) * kSampThreads + tid] = wt;
            sum.x += wt;
        }
        if (drow) {
            if (a.staged) {
                __syncthreads();  // everyone has read the target row
                stage_row(drow, true);
                __syncthreads();
            }
            for (int v = t_lo, i = 0; v < t_hi; ++v, ++i) {
                const float xd = a.staged ? s_stage[tid * (per_thr + 1) + i] : __ldg(drow + v);
                const double wd = exp(static_cast<double>(xd) * a.inv_t - mx_d);
                __stcg(Q + static_cast<int64_t>(i) * kSampThreads + tid, wd);
                sum.y += wd;
            }
        }
        publish_children(0, n_child);
        sum = cluster_reduce2<false>(sum, s_red, s_peer, set, rank);
        Pending pend = {1, recip_or_zero(sum.x), 0.0, -1};
        double sq = drow ? recip_or_zero(sum.y) : 0.0;  // draft side: q = Q * sq
        // One pass over this thread's tokens: bring P up to date in place (and retire the token the pending
        // round removed), hand the current (p, q) of each token to `f`.  The draft side is only read at
        // nodes that have children (`with_q`); a leaf has no draft row.
        auto pass = [&](bool with_q, auto&& f) {
            constexpr int kGroup = 4;  // draft-side values fetched together: their loads are in flight at once
            for (int v0 = t_lo, i0 = 0; v0 < t_hi; v0 += kGroup, i0 += kGroup) {
                double q_raw[kGroup];
#pragma unroll
                for (int u = 0; u < kGroup; ++u)
                    q_raw[u] = (with_q && v0 + u < t_hi) ? __ldcg(Q + static_cast<int64_t>(i0 + u) * kSampThreads + tid) : 0.0;
#pragma unroll
                for (int u = 0; u < kGroup; ++u) {
                    const int v = v0 + u;
                    if (v >= t_hi) break;
                    double* pp = P + static_cast<int64_t>(i0 + u) * kSampThreads + tid;
                    double p = *pp;
                    if (pend.kind) {
                        p = apply(pend, p, q_raw[u]);
                        *pp = p;
                        if (pend.kind == 2 && v == pend.x) {
                            __stcg(Q + static_cast<int64_t>(i0 + u) * kSampThreads + tid, 0.0);
                            q_raw[u] = 0.0;
                        }
                    }
                    f(v, p, q_raw[u] * sq);
                }
            }
        };
        // ---- try the children ---------------------------------------------------------------------
        int next = -1;
        for (int j = 0; j < n_child && j < a.max_k; ++j) {
            const int child = s_children[j];
            const int x = s_tok[child];
            if (tid == 0) {
                // (P, Q) of child j's token as the last pass left them, brought up to date here
                const double* at = table + ((j & 1) * RESPS_MAX_K + j) * 2;
                const double q_raw = __ldcg(at + 1);
                const double p = apply(pend, __ldcg(at), q_raw), q = q_raw * sq;
                const double alpha = q > 0.0 ? fmin(1.0, p / q) : (p > 0.0 ? 1.0 : 0.0);
                const double u = a.u_accept[(static_cast<int64_t>(b) * cap + acc) * a.max_k + j];
                s_decision = (u < alpha) ? child : -1;
            }
            __syncthreads();
            next = s_decision;
            if (next >= 0) break;
            // rejected: the residual's normaliser and the draft mass that is left without x
            Pair zr = {0.0, 0.0};
            pass(true, [&](int v, double p, double q) {
                zr.x += fmax(p - q, 0.0);
                if (v != x) zr.y += q;
            });
            publish_children((j + 1) & 1, n_child);
            zr = cluster_reduce2<false>(zr, s_red, s_peer, set, rank);
            pend = Pending{2, recip_or_zero(zr.x), sq, x};
            if (zr.y > 0.0) sq = sq * (1.0 / zr.y);
        }
        if (next >= 0) {
            cur = next;
            ++acc;
            if (rank == 0 && tid == 0) {
                a.accept_path[b * cap + acc] = cur;
                a.out_tokens[b * cap + acc - 1] = s_tok[cur];
            }
            continue;  // (the next node's first reduction is a cluster barrier before anything is overwritten)
        }
        // ---- nobody accepted (or a leaf): draw from the current target-side distribution --------------
        // inverse CDF in token order: this thread's run, the runs before it in the CTA, the CTAs before it
        double run = 0.0;
        pass(drow != nullptr, [&](int, double p, double) { run += p; });
        pend.kind = 0;
        // exclusive prefix of the runs over the CTA's threads
        const int lane = tid & 31, warp = tid >> 5;
        double inc = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double w = __shfl_up_sync(kFull, inc, o);
            if (lane >= o) inc += w;
        }
        __syncthreads();
        if (lane == 31) s_scan[warp] = inc;
        __syncthreads();
        double before = 0.0, cta_total = 0.0;
        for (int w = 0; w < kSampThreads / 32; ++w) {
            if (w < warp) before += s_scan[w];
            cta_total += s_scan[w];
        }
        const double excl = before + inc - run;
        if (tid < kClu) store_to_peer(&s_peer[set][rank][0], tid, cta_total);
        if (rank == 0 && tid == 0) __stcg(scratch + 4 * kClu, -1.0);
        cluster_barrier();
        double offset = 0.0, total = 0.0;
        for (int c = 0; c < kClu; ++c) {
            const double t = s_peer[set][c][0];
            if (c < static_cast<int>(rank)) offset += t;
            total += t;
        }
        set ^= 1;
        const double target = a.u_sample[static_cast<int64_t>(b) * cap + acc] * total;
        // the owner of the target: the last non-empty run that starts at or before it
        const double start = offset + excl;
        const bool last_run = (t_hi == V) && (t_lo < t_hi);
        if (t_lo < t_hi && start <= target && (start + run > target || last_run)) {
            double cum = start;
            int pick = t_hi - 1;
            for (int v = t_lo, i = 0; v < t_hi; ++v, ++i) {
                cum += P[static_cast<int64_t>(i) * kSampThreads + tid];  // (up to date since the pass above)
                if (cum > target) {
                    pick = v;
                    break;
                }
            }
            __stcg(scratch + 4 * kClu, static_cast<double>(pick));
        }
        cluster_barrier();
        if (rank == 0 && tid == 0) {
            int tok = static_cast<int>(__ldcg(scratch + 4 * kClu));
            if (tok < 0) tok = V - 1;  // rounding left the target past every run: the last token
            a.out_tokens[b * cap + acc] = tok;
            a.accept_len[b] = acc;
            if (a.steps_next) {
                resps_step s = a.steps[b];
                s.prefix_len += acc + 1;
                a.steps_next[b] = s;
            }
        }
        break;
    }
    cluster_barrier();  // nobody leaves while a peer may still be at the barrier before
}

}  // namespace

constexpr size_t kDynSmemCap = 220 * 1024;
static int sampled_per_thr(int vocab) {
    const int per_cta = (vocab + kClu - 1) / kClu;
    return (per_cta + kSampThreads - 1) / kSampThreads;
}
static size_t sampled_stage_bytes(int vocab) {  // one row's slice, padded rows
    return sizeof(float) * kSampThreads * static_cast<size_t>(sampled_per_thr(vocab) + 1);
}
static size_t sampled_p_bytes(int vocab) { return sizeof(double) * kSampThreads * static_cast<size_t>(sampled_per_thr(vocab)); }

cudaError_t sampled_setup(resps_ctx*) {
    return cudaFuncSetAttribute(accept_sampled_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                static_cast<int>(kDynSmemCap));
}

static int64_t sampled_state_per_cta(int vocab) {
    const int per_cta = (vocab + kClu - 1) / kClu;
    const int per_thr = (per_cta + kSampThreads - 1) / kSampThreads;
    return static_cast<int64_t>(per_thr) * kSampThreads;
}

size_t sampled_scratch_doubles(int max_batch, int vocab) {
    return static_cast<size_t>(max_batch) * (kScratchPerSeq + kClu * 2 * sampled_state_per_cta(vocab));
}

cudaError_t launch_accept_sampled(const resps_ctx* ctx, const resps_step* d_steps, const int32_t* d_n_nodes, int batch,
                                  const float* target, int64_t ld_b, int64_t ld_row, const float* draft, int64_t dld_b,
                                  int64_t dld_level, int64_t dld_row, double temperature, const int32_t* tokens,
                                  const int32_t* parent, const double* u_accept, const double* u_sample,
                                  int32_t* accept_path, int32_t* accept_len, int32_t* out_tokens, resps_step* steps_next,
                                  cudaStream_t st) {
    SampledArgs a;
    a.steps = d_steps, a.n_nodes = d_n_nodes;
    a.target = target, a.ld_b = ld_b, a.ld_row = ld_row;
    a.draft = draft, a.dld_b = dld_b, a.dld_level = dld_level, a.dld_row = dld_row;
    a.node_row = ctx->ws.node_row;
    a.temperature = temperature, a.inv_t = 1.0 / temperature;
    a.tokens = tokens, a.parent = parent, a.u_accept = u_accept, a.u_sample = u_sample;
    a.vocab = ctx->shape.vocab, a.max_tt = ctx->shape.max_tt, a.max_depth = ctx->shape.max_depth;
    a.max_k = ctx->shape.max_k;
    a.accept_path = accept_path, a.accept_len = accept_len, a.out_tokens = out_tokens, a.steps_next = steps_next;
    a.scratch = ctx->ws.samp_scratch;
    a.state_per_cta = sampled_state_per_cta(ctx->shape.vocab);
    const size_t stage_bytes = sampled_stage_bytes(ctx->shape.vocab), p_bytes = sampled_p_bytes(ctx->shape.vocab);
    a.p_in_smem = (p_bytes + stage_bytes <= kDynSmemCap) ? 1 : 0;
    a.staged = ((a.p_in_smem ? p_bytes : 0) + stage_bytes <= kDynSmemCap) ? 1 : 0;
    const size_t dyn_bytes = (a.p_in_smem ? p_bytes : 0) + (a.staged ? stage_bytes : 0);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(batch * kClu), cfg.blockDim = dim3(kSampThreads), cfg.dynamicSmemBytes = dyn_bytes, cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = kClu, attr[1].val.clusterDim.y = 1, attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr, cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, accept_sampled_kernel, a);
}

}  // namespace resps
