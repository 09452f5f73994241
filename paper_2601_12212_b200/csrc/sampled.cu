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
// vocabulary, partial sums meet through a few words of global memory behind the hardware cluster
// barrier (no spinning anywhere), and every CTA then takes the same decision from the same numbers.
// Arithmetic is fp64 throughout: a decision (accept or not, which token) is a comparison of sums over
// 10^5 terms, and only at fp64 is the order of summation immaterial to it.
#include <cmath>

#include "common.cuh"

namespace resps {
namespace {

constexpr int kClu = 8;             // CTAs per sequence
constexpr int kSampThreads = 1024;
constexpr int kMaxRounds = RESPS_MAX_K;  // rejected siblings at one node
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
    double* scratch;  // [batch][kScratchPerSeq]
};
constexpr int kScratchPerSeq = 2 * kClu + 8;  // two alternating sets of partials, then the drawn token

__device__ __forceinline__ unsigned cluster_rank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Sum (or maximum) over the CTA, result in every thread.
template <bool MAX>
__device__ __forceinline__ double block_reduce(double v, double* s_red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double w = __shfl_xor_sync(kFull, v, o);
        v = MAX ? fmax(v, w) : v + w;
    }
    __syncthreads();  // s_red is free again
    if (lane == 0) s_red[warp] = v;
    __syncthreads();
    double r = s_red[0];
    for (int w = 1; w < kSampThreads / 32; ++w) r = MAX ? fmax(r, s_red[w]) : r + s_red[w];
    return r;
}

// The same over the cluster: the CTAs' results meet in global memory behind the cluster barrier and
// every thread adds them up in rank order, so all CTAs hold the same bits.  `set` alternates between
// consecutive reductions (a set is written again only after everyone has read it).
template <bool MAX>
__device__ __forceinline__ double cluster_reduce(double v, double* s_red, double* scratch, int& set, unsigned rank) {
    const double mine = block_reduce<MAX>(v, s_red);
    double* slot = scratch + set * kClu;
    if (threadIdx.x == 0) __stcg(slot + rank, mine);
    cluster_barrier();
    double r = __ldcg(slot);
    for (int c = 1; c < kClu; ++c) r = MAX ? fmax(r, __ldcg(slot + c)) : r + __ldcg(slot + c);
    set ^= 1;
    return r;
}

__global__ void __launch_bounds__(kSampThreads, 1) accept_sampled_kernel(const SampledArgs a) {
    pdl_wait();  // the kernel before this one in the stream has completed
    pdl_launch_dependents();
    __shared__ double s_red[kSampThreads / 32];
    __shared__ double s_scan[kSampThreads / 32];
    __shared__ int s_tok[RESPS_MAX_TT], s_par[RESPS_MAX_TT];
    __shared__ int s_children[RESPS_MAX_TT];
    __shared__ int s_removed[kMaxRounds];       // tokens of the rejected siblings, in order
    __shared__ double s_z[kMaxRounds];          // normaliser of the residual after each rejection (0: residual kept)
    __shared__ double s_rest[kMaxRounds];       // draft mass left after each removal
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
        // ---- P_T(. | cur) = softmax(row / T): maximum, then the sum of exponentials ------------------
        float fm = -INFINITY;
        for (int v = t_lo; v < t_hi; ++v) fm = fmaxf(fm, __ldg(trow + v));
        const double mx_t = cluster_reduce<true>(static_cast<double>(fm), s_red, scratch, set, rank) * a.inv_t;
        double sum = 0.0;
        for (int v = t_lo; v < t_hi; ++v) sum += exp(static_cast<double>(__ldg(trow + v)) * a.inv_t - mx_t);
        const double s_t = cluster_reduce<false>(sum, s_red, scratch, set, rank);
        const int n_child = s_nchild;  // (the reductions above synchronised the CTA)
        const float* drow = nullptr;
        double mx_d = 0.0, s_d = 1.0;
        if (n_child > 0) {
            const int row = a.node_row[ob + cur];  // >= 0 for a node with children
            drow = a.draft + b * a.dld_b + (row / RESPS_MAX_K) * a.dld_level + (row % RESPS_MAX_K) * a.dld_row;
            fm = -INFINITY;
            for (int v = t_lo; v < t_hi; ++v) fm = fmaxf(fm, __ldg(drow + v));
            mx_d = cluster_reduce<true>(static_cast<double>(fm), s_red, scratch, set, rank) * a.inv_t;
            sum = 0.0;
            for (int v = t_lo; v < t_hi; ++v) sum += exp(static_cast<double>(__ldg(drow + v)) * a.inv_t - mx_d);
            s_d = cluster_reduce<false>(sum, s_red, scratch, set, rank);
        }
        // p and q of one token after `rounds` rejections at this node
        auto eval = [&](int v, int rounds, double& p, double& q) {
            p = exp(static_cast<double>(__ldg(trow + v)) * a.inv_t - mx_t) / s_t;
            q = drow ? exp(static_cast<double>(__ldg(drow + v)) * a.inv_t - mx_d) / s_d : 0.0;
            for (int i = 0; i < rounds; ++i) {
                if (s_z[i] > 0.0) p = fmax(p - q, 0.0) / s_z[i];
                q = (v == s_removed[i]) ? 0.0 : (s_rest[i] > 0.0 ? q / s_rest[i] : q);
            }
        };
        // ---- try the children ---------------------------------------------------------------------
        int rounds = 0, next = -1;
        for (int j = 0; j < n_child && j < a.max_k; ++j) {
            const int child = s_children[j];
            const int x = s_tok[child];
            if (tid == 0) {
                double p, q;
                eval(x, rounds, p, q);
                const double alpha = q > 0.0 ? fmin(1.0, p / q) : (p > 0.0 ? 1.0 : 0.0);
                const double u = a.u_accept[(static_cast<int64_t>(b) * cap + acc) * a.max_k + j];
                s_decision = (u < alpha) ? child : -1;
            }
            __syncthreads();
            next = s_decision;
            if (next >= 0) break;
            // rejected: the residual's normaliser and the draft mass that is left without x
            double z = 0.0, rest = 0.0;
            for (int v = t_lo; v < t_hi; ++v) {
                double p, q;
                eval(v, rounds, p, q);
                z += fmax(p - q, 0.0);
                if (v != x) rest += q;
            }
            z = cluster_reduce<false>(z, s_red, scratch, set, rank);
            rest = cluster_reduce<false>(rest, s_red, scratch, set, rank);
            if (tid == 0) s_removed[rounds] = x, s_z[rounds] = z, s_rest[rounds] = rest;
            __syncthreads();
            ++rounds;
        }
        if (next >= 0) {
            cur = next;
            ++acc;
            if (rank == 0 && tid == 0) {
                a.accept_path[b * cap + acc] = cur;
                a.out_tokens[b * cap + acc - 1] = s_tok[cur];
            }
            continue;
        }
        // ---- nobody accepted (or a leaf): draw from the current target-side distribution --------------
        // inverse CDF in token order: this thread's run, the runs before it in the CTA, the CTAs before it
        double run = 0.0;
        for (int v = t_lo; v < t_hi; ++v) {
            double p, q;
            eval(v, rounds, p, q);
            run += p;
        }
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
        double* slot = scratch + set * kClu;
        if (tid == 0) __stcg(slot + rank, cta_total);
        if (rank == 0 && tid == 0) __stcg(scratch + 2 * kClu, -1.0);
        cluster_barrier();
        double offset = 0.0, total = 0.0;
        for (int c = 0; c < kClu; ++c) {
            const double t = __ldcg(slot + c);
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
            for (int v = t_lo; v < t_hi; ++v) {
                double p, q;
                eval(v, rounds, p, q);
                cum += p;
                if (cum > target) {
                    pick = v;
                    break;
                }
            }
            __stcg(scratch + 2 * kClu, static_cast<double>(pick));
        }
        cluster_barrier();
        if (rank == 0 && tid == 0) {
            int tok = static_cast<int>(__ldcg(scratch + 2 * kClu));
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

size_t sampled_scratch_doubles(int max_batch) { return static_cast<size_t>(max_batch) * kScratchPerSeq; }

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
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(batch * kClu), cfg.blockDim = dim3(kSampThreads), cfg.dynamicSmemBytes = 0, cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = kClu, attr[1].val.clusterDim.y = 1, attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr, cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, accept_sampled_kernel, a);
}

}  // namespace resps
