// Re-SpS speculative-step ORACLE  --  TEST INFRASTRUCTURE, NOT THE PRODUCT.
//
// A plain, slow, single-threaded fp64 CPU statement of what one speculative
// step computes (draft-tree construction, tree-masked attention, greedy
// verification, KV-cache compaction).  It exists so that the CUDA library can
// be checked against something that can be compared with the paper by eye.
// Only tests, the smoke check and the benchmark's CPU-baseline leg may call it;
// it shares no source, header, table or helper with the CUDA path.
//
// Every function is a definition written out (full ordering, naive softmax),
// or the paper's algorithm taken step by step; there is no blocking, fusion or
// reordering.  Pins (what each function is checked against, see tests/):
//   top-k / argmax : brute-force full sort, k=1 == argmax, k=V == sort,
//                    library top-k on distinct values
//   lse / scores   : closed forms (uniform row, dominant row), sum of probs = 1
//   tree           : structural invariants, k=1 chain, d=1 star, exhaustive
//                    brute force over all root paths on tiny inputs
//   attention      : chain tree == causal attention (library routine),
//                    one-node tree == plain decode, closed forms, poison slots
//   accept         : brute force over retrieve rows, chain == longest common prefix
//   sampled accept : chain of sampled draft tokens keeps the target's distribution (chi-square
//                    against the exact P_T, acceptance rate = sum min(p, q)); T -> 0 equals greedy
//   compaction     : gather definition, identity path is a no-op
//   whole step     : greedy speculative decoding over a tiny random transformer
//                    reproduces greedy autoregressive decoding token for token
// Parity unpinned (conventions of this implementation that no external value fixes):
//   the tie-break orders (equal logits -> lower token id, equal scores -> lower
//   candidate index), the node order (ascending candidate index), the retrieve
//   row order, reading "depth d" as d draft levels, and -- in the sampled
//   acceptance -- how the siblings of a tree are tried after a rejection (the paper
//   gives the rule for a chain only).
//
// Build: g++ -O2 -std=c++17 -shared -fPIC resps_oracle.cpp -o libresps_oracle.so

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

namespace {

// bf16 -> fp64, exact (bf16 is the top 16 bits of an IEEE fp32).
inline double bf16_to_f64(uint16_t h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

struct ValId {
    float v;
    int32_t id;
};
// Total order used for vocabulary selection: larger value first, equal values
// by smaller token id.
inline bool val_before(const ValId& a, const ValId& b) {
    if (a.v != b.v) return a.v > b.v;
    return a.id < b.id;
}

struct ScoreIdx {
    double s;
    int32_t c;
};
// Total order used for candidate selection: larger cumulative score first,
// equal scores by smaller candidate index (a parent always precedes its child).
inline bool score_before(const ScoreIdx& a, const ScoreIdx& b) {
    if (a.s != b.s) return a.s > b.s;
    return a.c < b.c;
}

// Section 3.2, "Draft Tree Expansion": the k most confident tokens of one draft
// distribution, and log-sum-exp of the row (so that confidence c = softmax prob
// and log c = x - lse).
void topk_lse_row(const float* row, int V, int k, ValId* out, double* lse) {
    std::vector<ValId> all(V);
    for (int v = 0; v < V; ++v) all[v] = ValId{row[v], v};
    std::partial_sort(all.begin(), all.begin() + k, all.end(), val_before);
    for (int r = 0; r < k; ++r) out[r] = all[r];
    double mx = -std::numeric_limits<double>::infinity();
    for (int v = 0; v < V; ++v) mx = std::max(mx, static_cast<double>(row[v]));
    double sum = 0.0;
    for (int v = 0; v < V; ++v) sum += std::exp(static_cast<double>(row[v]) - mx);
    *lse = mx + std::log(sum);
}

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------
// Vocabulary top-k with log-sum-exp for one row (Section 3.2, Draft Tree
// Expansion; Algorithm 2, the "select highest children" step).
// ---------------------------------------------------------------------------
int oracle_topk_lse(const float* row, int V, int k, float* out_val, int32_t* out_id,
                    double* out_lse) {
    if (V < 1 || k < 1 || k > V) return -1;
    std::vector<ValId> top(k);
    double lse;
    topk_lse_row(row, V, k, top.data(), &lse);
    for (int r = 0; r < k; ++r) {
        out_val[r] = top[r].v;
        out_id[r] = top[r].id;
    }
    *out_lse = lse;
    return 0;
}

// ---------------------------------------------------------------------------
// Draft-tree construction for one sequence (Section 3.2, Draft Tree Expansion
// and Confidence-Based Candidate Reranking; Algorithm 2, tree-building loop and
// rerank).
//
// logits[level][slot][V] (fp32, strides ld_level / ld_row in elements): the
// draft model's output for the slot-th frontier node of that level; level 0
// uses slot 0 only (the root's distribution).
//
// Readings taken where the paper is silent or inconsistent:
//  * TT counts the root; d is the number of draft levels (node depths 1..d);
//    all d levels are always expanded and TT only caps the rerank.
//  * V_i is kept as a sum of log-probabilities.
//  * n = min(TT, 1 + n_cand): the hyper-parameters are upper limits.
//
// Outputs (caller-allocated, capacities max_tt / max_tt*(ret_stride)):
//   tokens, parent (root = -1), depth, position_ids = L + depth,
//   mask[i][2] (bit j of the 128-bit word  <=>  node j is i or an ancestor of i),
//   retrieve[row][ret_stride] (root-to-leaf node indices, -1 padded),
//   n_leaves, n_nodes,
//   cand_score[n_cand], cand_token[n_cand], cand_parent[n_cand] (optional, may be
//   null): cumulative log-prob, token and parent candidate (-1 = root) of every
//   expanded child, candidate c = k + (j-1)k^2 + p*k + r for level j >= 1,
//   frontier[d][k] (optional): the candidates chosen for expansion after each
//   level (row j = the frontier whose draft rows are logits[j+1][.]),
//   min_gap (optional): smallest fp64 score gap across any selection boundary; +inf if
//   none.  The boundaries are the pairs of neighbours in score order whose order
//   decides the result: among the k+1 best of a level that is expanded further
//   (levels 1..d-2: the rank inside the frontier is the slot whose draft row the
//   node is given, the (k+1)-th is the first one left out; level 0 is ordered by
//   the raw logits of one row, which is exact), and the m-th vs the (m+1)-th of
//   the rerank.
//
// Near ties (test support for implementations whose log-sum-exp is summed in another
// order and may therefore resolve a gap below `tau` the other way):
//   near_pairs (optional, capacity max_near pairs): every boundary pair (before,
//   after) as above whose gap is below tau; n_near = their number.
//   node_cand (optional, [max_tt]): the candidate index each node was made from (-1 for the
//   root); with frontier[][] it tells which draft row a node's children were taken from.
//   order_bias (optional, [n_cand]): added to a candidate's score where candidates
//   are *ordered* (frontier choice and rerank), never to the score its children
//   inherit.  A bias that lifts `after` just above `before` yields the tree of the
//   swapped order, i.e. the result "up to a swap among candidates within tau".
// ---------------------------------------------------------------------------
int oracle_tree_expand(int32_t root_token, const float* logits, int64_t ld_level, int64_t ld_row,
                       int V, int TT, int d, int k, int L, int max_tt, int ret_stride,
                       int32_t* tokens, int32_t* parent, int32_t* depth, int32_t* position_ids,
                       uint64_t* mask, int32_t* retrieve, int32_t* n_leaves, int32_t* n_nodes,
                       double* cand_score, int32_t* cand_token, int32_t* cand_parent,
                       int32_t* frontier_out, double* min_gap, const double* order_bias, double tau,
                       int32_t* near_pairs, int max_near, int32_t* n_near, int32_t* node_cand) {
    if (V < 1 || k < 1 || k > V || d < 1 || TT < 1 || TT > max_tt || max_tt > 128) return -1;
    if (ret_stride < d + 1) return -1;
    const int n_cand = k + (d - 1) * k * k;
    std::vector<int32_t> c_tok(n_cand), c_par(n_cand), c_dep(n_cand);
    std::vector<double> c_score(n_cand);
    double gap = std::numeric_limits<double>::infinity();
    int near = 0;
    auto boundary = [&](const ScoreIdx& before, const ScoreIdx& after) {
        const double g = before.s - after.s;
        gap = std::min(gap, g);
        if (g < tau && near_pairs && near < max_near) {
            near_pairs[2 * near + 0] = before.c;
            near_pairs[2 * near + 1] = after.c;
            ++near;
        }
    };
    auto ordering_score = [&](double s, int c) { return order_bias ? s + order_bias[c] : s; };
    std::vector<ValId> top(k);
    double lse;

    // Level 0: children of the root.
    topk_lse_row(logits, V, k, top.data(), &lse);
    for (int r = 0; r < k; ++r) {
        c_tok[r] = top[r].id;
        c_par[r] = -1;  // ROOT
        c_dep[r] = 1;
        c_score[r] = static_cast<double>(top[r].v) - lse;
    }
    std::vector<int32_t> frontier(k);
    for (int r = 0; r < k; ++r) frontier[r] = r;
    if (frontier_out)
        for (int r = 0; r < k; ++r) frontier_out[r] = r;

    // Levels 1..d-1: expand each frontier node, then pick the next frontier as
    // the k best of the whole layer by cumulative score.
    for (int j = 1; j < d; ++j) {
        const int base = k + (j - 1) * k * k;
        for (int p = 0; p < k; ++p) {
            const float* row = logits + j * ld_level + p * ld_row;
            topk_lse_row(row, V, k, top.data(), &lse);
            for (int r = 0; r < k; ++r) {
                const int c = base + p * k + r;
                c_tok[c] = top[r].id;
                c_par[c] = frontier[p];
                c_dep[c] = j + 1;
                c_score[c] = c_score[frontier[p]] + (static_cast<double>(top[r].v) - lse);
            }
        }
        std::vector<ScoreIdx> layer(k * k);
        for (int i = 0; i < k * k; ++i) layer[i] = ScoreIdx{ordering_score(c_score[base + i], base + i), base + i};
        std::sort(layer.begin(), layer.end(), score_before);
        for (int r = 0; r < k; ++r) frontier[r] = layer[r].c;
        if (frontier_out)
            for (int r = 0; r < k; ++r) frontier_out[j * k + r] = frontier[r];
        if (j + 1 < d)  // this frontier is expanded: its members and their order matter
            for (int r = 0; r < k && r + 1 < k * k; ++r) boundary(layer[r], layer[r + 1]);
    }

    // Rerank every candidate; keep the best m, in candidate order.
    const int m = std::min(TT - 1, n_cand);
    std::vector<ScoreIdx> all(n_cand);
    for (int c = 0; c < n_cand; ++c) all[c] = ScoreIdx{ordering_score(c_score[c], c), c};
    std::sort(all.begin(), all.end(), score_before);
    if (m >= 1 && m < n_cand) boundary(all[m - 1], all[m]);
    std::vector<int32_t> kept(m);
    for (int i = 0; i < m; ++i) kept[i] = all[i].c;
    std::sort(kept.begin(), kept.end());

    // Emit nodes: node 0 is the root, node i+1 is the i-th kept candidate.
    const int n = m + 1;
    std::vector<int32_t> node_of_cand(n_cand, -1);
    for (int i = 0; i < m; ++i) node_of_cand[kept[i]] = i + 1;
    if (node_cand) {
        node_cand[0] = -1;
        for (int i = 0; i < m; ++i) node_cand[i + 1] = kept[i];
    }
    tokens[0] = root_token;
    parent[0] = -1;
    depth[0] = 0;
    position_ids[0] = L;
    mask[0] = 1ull;
    mask[1] = 0ull;
    for (int i = 1; i < n; ++i) {
        const int c = kept[i - 1];
        tokens[i] = c_tok[c];
        const int pn = (c_par[c] < 0) ? 0 : node_of_cand[c_par[c]];
        if (pn < 0) return -2;  // kept set not ancestor-closed: cannot happen with these orders
        parent[i] = pn;
        depth[i] = c_dep[c];
        position_ids[i] = L + c_dep[c];
        mask[2 * i + 0] = mask[2 * pn + 0];
        mask[2 * i + 1] = mask[2 * pn + 1];
        mask[2 * i + (i >> 6)] |= (1ull << (i & 63));
    }

    // Retrieve rows: one per leaf, ascending leaf index, root first.
    std::vector<char> has_child(n, 0);
    for (int i = 1; i < n; ++i) has_child[parent[i]] = 1;
    int rows = 0;
    for (int i = 0; i < n; ++i) {
        if (has_child[i]) continue;
        int32_t* row = retrieve + static_cast<int64_t>(rows) * ret_stride;
        for (int t = 0; t < ret_stride; ++t) row[t] = -1;
        int len = depth[i] + 1;
        int cur = i;
        for (int t = len - 1; t >= 0; --t) {
            row[t] = cur;
            cur = parent[cur];
        }
        ++rows;
    }
    *n_leaves = rows;
    *n_nodes = n;
    for (int c = 0; c < n_cand; ++c) {
        if (cand_score) cand_score[c] = c_score[c];
        if (cand_token) cand_token[c] = c_tok[c];
        if (cand_parent) cand_parent[c] = c_par[c];
    }
    if (min_gap) *min_gap = gap;
    if (n_near) *n_near = near;
    return 0;
}

// ---------------------------------------------------------------------------
// Tree-masked verification attention for one sequence and one layer
// (Section 3.2, Verification Phase: the target scores every tree token in one
// pass; Appendix D: attention masks adjusted to the tree).
//
// q      bf16 [n][Hq][D]
// k,v    bf16 cache [Hkv][capacity][D] given by element strides; the tree tokens'
//        K/V already sit at slots L .. L+n-1
// mask   [n][2] uint64, ancestor-or-self bits
// out    fp64 [n][Hq][D];  lse (optional) fp64 [n][Hq] = log sum_j exp(s_j)
//
// Node t may see cache slots 0..L-1 and slot L+j for every set bit j of mask[t].
// No other slot is read.
// ---------------------------------------------------------------------------
int oracle_tree_attention(int n, int Hq, int Hkv, int D, int L, const uint16_t* q,
                          const uint16_t* k_cache, const uint16_t* v_cache, int64_t stride_head,
                          int64_t stride_tok, const uint64_t* mask, double scale, double* out,
                          double* lse_out) {
    if (n < 1 || n > 128 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
    std::vector<int> allowed;
    std::vector<double> s;
    for (int t = 0; t < n; ++t) {
        allowed.clear();
        for (int j = 0; j < L; ++j) allowed.push_back(j);
        for (int j = 0; j < n; ++j)
            if ((mask[2 * t + (j >> 6)] >> (j & 63)) & 1ull) allowed.push_back(L + j);
        for (int h = 0; h < Hq; ++h) {
            const int g = h / G;
            const uint16_t* qv = q + (static_cast<int64_t>(t) * Hq + h) * D;
            s.assign(allowed.size(), 0.0);
            double mx = -std::numeric_limits<double>::infinity();
            for (size_t a = 0; a < allowed.size(); ++a) {
                const uint16_t* kv = k_cache + g * stride_head + allowed[a] * stride_tok;
                double dot = 0.0;
                for (int e = 0; e < D; ++e) dot += bf16_to_f64(qv[e]) * bf16_to_f64(kv[e]);
                s[a] = dot * scale;
                mx = std::max(mx, s[a]);
            }
            double denom = 0.0;
            for (size_t a = 0; a < allowed.size(); ++a) {
                s[a] = std::exp(s[a] - mx);
                denom += s[a];
            }
            double* o = out + (static_cast<int64_t>(t) * Hq + h) * D;
            for (int e = 0; e < D; ++e) o[e] = 0.0;
            for (size_t a = 0; a < allowed.size(); ++a) {
                const uint16_t* vv = v_cache + g * stride_head + allowed[a] * stride_tok;
                for (int e = 0; e < D; ++e) o[e] += s[a] * bf16_to_f64(vv[e]);
            }
            for (int e = 0; e < D; ++e) o[e] /= denom;
            if (lse_out) lse_out[static_cast<int64_t>(t) * Hq + h] = mx + std::log(denom);
        }
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Greedy verification and acceptance for one sequence (Section 3.1 greedy rule;
// Section 3.2 Acceptance Criterion at temperature 0: a draft token is accepted
// iff it equals the target's argmax at its parent; Algorithm 2 "get accepted
// tokens").
//
// target_logits fp32 [n][V] (row stride ld_row): target distribution after node i.
// Outputs: target_argmax[n] (ties -> lowest id); accept_path[a+1] node indices
// with path[0] = 0 (unused entries up to path_cap set to -1); accept_len = a;
// out_tokens[a+1] = the a accepted draft tokens followed by the bonus token
// (target argmax at the last accepted node); unused entries -1.
// ---------------------------------------------------------------------------
int oracle_verify_accept(int n, int V, const float* target_logits, int64_t ld_row,
                         const int32_t* tokens, const int32_t* parent, int path_cap,
                         int32_t* target_argmax, int32_t* accept_path, int32_t* accept_len,
                         int32_t* out_tokens) {
    if (n < 1 || V < 1) return -1;
    for (int i = 0; i < n; ++i) {
        const float* row = target_logits + i * ld_row;
        int best = 0;
        for (int v = 1; v < V; ++v)
            if (row[v] > row[best]) best = v;
        target_argmax[i] = best;
    }
    for (int t = 0; t < path_cap; ++t) {
        accept_path[t] = -1;
        out_tokens[t] = -1;
    }
    int cur = 0, a = 0;
    accept_path[0] = 0;
    for (;;) {
        int next = -1;
        for (int c = 1; c < n; ++c)
            if (parent[c] == cur && tokens[c] == target_argmax[cur]) {
                next = c;
                break;
            }
        if (next < 0) break;
        if (a + 1 >= path_cap) return -2;
        cur = next;
        ++a;
        accept_path[a] = cur;
        out_tokens[a - 1] = tokens[cur];
    }
    out_tokens[a] = target_argmax[cur];
    *accept_len = a;
    return 0;
}

// ---------------------------------------------------------------------------
// Verification and acceptance under sampling (temperature T > 0) for one sequence
// (Section 3.2, "Acceptance Criterion": a draft token y is accepted with probability
// alpha = min(1, P_T(y | .) / P_d(y | .)); Section 4.1, "Lossless Output Fidelity":
// speculative sampling with rejection-based correction keeps the target's output
// distribution).
//
// P_T(. | node i) = softmax(target_logits[i] / T); P_d(. | node i) = softmax(draft
// row of node i / T), the row its children were taken from (node_row[i], -1 for a node
// that was not expanded).  All arithmetic in fp64.
//
// The paper states the rule for a chain of draft tokens.  For a chain this function is
// that rule, with the correction step of the speculative-sampling papers it cites: on
// the first rejected token the emitted token is drawn from the normalised residual
// max(0, P_T - P_d); after the last accepted token of a chain that was accepted in full
// it is drawn from P_T.  Reading for a tree (the paper is silent): the children of the
// current node are tried in node order (= the draft's order of preference); after a
// rejected child x the target-side distribution becomes the normalised residual
// max(0, p - q) and the draft-side one q with x removed, renormalised, and the next
// sibling is tried against those; when no child is left the token is drawn from the
// residual.  (A residual that is zero everywhere leaves p as it is.)
//
// Random numbers are inputs: u_accept[level * max_children + j] for the j-th child tried
// at walk level `level`, u_sample[level] for the token drawn when the walk stops there;
// all uniform in (0, 1).  A token is drawn by inverse CDF in token-id order: the first v
// with sum_{w <= v} p[w] > u * sum_w p[w].
//
// Outputs as oracle_verify_accept (path, accept_len, out_tokens; no argmax), and
// min_margin: the smallest distance of any decision from flipping -- |u - alpha| of
// every acceptance test that was taken with alpha < 1 or u near 1, and the distance of
// u * total from the two cumulative sums that bracket the drawn token, relative to
// total.  An implementation that sums in another order must reproduce every decision
// whose margin exceeds its own rounding error.
// ---------------------------------------------------------------------------
int oracle_verify_accept_sampled(int n, int V, const float* target_logits, int64_t ld_row,
                                 const float* draft_logits, int64_t draft_ld_row, const int32_t* node_row,
                                 const int32_t* tokens, const int32_t* parent, double temperature,
                                 const double* u_accept, int max_children, const double* u_sample,
                                 int path_cap, int32_t* accept_path, int32_t* accept_len,
                                 int32_t* out_tokens, double* min_margin) {
    if (n < 1 || V < 1 || !(temperature > 0.0) || path_cap < 1) return -1;
    auto softmax_t = [&](const float* row, std::vector<double>& out) {
        double mx = -std::numeric_limits<double>::infinity();
        for (int v = 0; v < V; ++v) mx = std::max(mx, static_cast<double>(row[v]) / temperature);
        double sum = 0.0;
        for (int v = 0; v < V; ++v) {
            out[v] = std::exp(static_cast<double>(row[v]) / temperature - mx);
            sum += out[v];
        }
        for (int v = 0; v < V; ++v) out[v] /= sum;
    };
    double margin = std::numeric_limits<double>::infinity();
    auto draw = [&](const std::vector<double>& p, double u) {
        double total = 0.0;
        for (int v = 0; v < V; ++v) total += p[v];
        const double target = u * total;
        double run = 0.0;
        for (int v = 0; v < V; ++v) {
            const double before = run;
            run += p[v];
            if (run > target || v == V - 1) {
                margin = std::min(margin, (target - before) / total);
                if (v < V - 1) margin = std::min(margin, (run - target) / total);
                return v;
            }
        }
        return V - 1;
    };
    for (int t = 0; t < path_cap; ++t) {
        accept_path[t] = -1;
        out_tokens[t] = -1;
    }
    std::vector<double> p(V), q(V);
    int cur = 0, a = 0;
    accept_path[0] = 0;
    for (;;) {
        softmax_t(target_logits + cur * ld_row, p);
        std::vector<int> children;
        for (int c = 1; c < n; ++c)
            if (parent[c] == cur) children.push_back(c);
        int next = -1;
        if (!children.empty()) {
            if (node_row[cur] < 0) return -3;  // a node with children must have a draft row
            softmax_t(draft_logits + node_row[cur] * draft_ld_row, q);
            for (size_t j = 0; j < children.size(); ++j) {
                if (static_cast<int>(j) >= max_children) return -4;
                const int x = tokens[children[j]];
                // (a draft probability that has underflowed to zero: the ratio is infinite, or 0/0 = reject)
                const double alpha = q[x] > 0.0 ? std::min(1.0, p[x] / q[x]) : (p[x] > 0.0 ? 1.0 : 0.0);
                const double u = u_accept[a * max_children + j];
                margin = std::min(margin, alpha < 1.0 ? std::fabs(u - alpha) : 1.0 - u);
                if (u < alpha) {
                    next = children[j];
                    break;
                }
                // rejected: residual on the target side, x removed on the draft side
                double z = 0.0;
                for (int v = 0; v < V; ++v) z += std::max(p[v] - q[v], 0.0);
                if (z > 0.0)
                    for (int v = 0; v < V; ++v) p[v] = std::max(p[v] - q[v], 0.0) / z;
                q[x] = 0.0;
                double rest = 0.0;  // (summed, not 1 - q[x]: a dominant q[x] rounds to 1 and would leave nothing)
                for (int v = 0; v < V; ++v) rest += q[v];
                if (rest > 0.0)
                    for (int v = 0; v < V; ++v) q[v] /= rest;
            }
        }
        if (next < 0) {
            out_tokens[a] = draw(p, u_sample[a]);
            break;
        }
        if (a + 1 >= path_cap) return -2;
        cur = next;
        ++a;
        accept_path[a] = cur;
        out_tokens[a - 1] = tokens[cur];
    }
    *accept_len = a;
    if (min_margin) *min_margin = margin;
    return 0;
}

// ---------------------------------------------------------------------------
// KV-cache compaction for one sequence and one layer (Appendix D, input update:
// rejected tokens are discarded from the cache).  Out-of-place definition:
// new[L+j] = old[L+path[j]] for j = 0..a, for K and V and every KV head; the
// new prefix length is L + a + 1.  Applied to the caller's buffers through a
// private copy of the old contents, so that it is a pure gather.
// ---------------------------------------------------------------------------
int oracle_kv_compact(int Hkv, int D, int L, const int32_t* accept_path, int accept_len,
                      uint16_t* k_cache, uint16_t* v_cache, int64_t stride_head,
                      int64_t stride_tok, int64_t n_elems) {
    std::vector<uint16_t> old_k(k_cache, k_cache + n_elems), old_v(v_cache, v_cache + n_elems);
    for (int g = 0; g < Hkv; ++g)
        for (int j = 0; j <= accept_len; ++j) {
            const int64_t dst = g * stride_head + static_cast<int64_t>(L + j) * stride_tok;
            const int64_t src = g * stride_head + static_cast<int64_t>(L + accept_path[j]) * stride_tok;
            if (dst + D > n_elems || src + D > n_elems) return -1;
            for (int e = 0; e < D; ++e) {
                k_cache[dst + e] = old_k[src + e];
                v_cache[dst + e] = old_v[src + e];
            }
        }
    return 0;
}

}  // extern "C"
