"""CPU oracle for the Re-SpS speculative step -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Thin numpy/ctypes wrapper over ``resps_oracle.cpp`` (single-threaded fp64 C++).
Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library never does, and the two share no code.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "resps_oracle.cpp")
_LIB = os.path.join(_HERE, "libresps_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, no OpenMP, no SIMD flags)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def topk_lse(row: np.ndarray, k: int):
    """Top-k (value desc, id asc) and log-sum-exp of one fp32 row."""
    row = _c(row, np.float32)
    V = row.shape[0]
    val = np.empty(k, np.float32)
    idx = np.empty(k, np.int32)
    lse = ctypes.c_double()
    rc = _load().oracle_topk_lse(_p(row), V, k, _p(val), _p(idx), ctypes.byref(lse))
    if rc != 0:
        raise ValueError(f"oracle_topk_lse rc={rc}")
    return val, idx, lse.value


@dataclass
class Tree:
    tokens: np.ndarray        # int32 [n]
    parent: np.ndarray        # int32 [n], root -1
    depth: np.ndarray         # int32 [n]
    position_ids: np.ndarray  # int32 [n]
    mask: np.ndarray          # uint64 [n, 2]
    retrieve: np.ndarray      # int32 [n_leaves, ret_stride]
    n_nodes: int
    n_leaves: int
    cand_score: np.ndarray    # float64 [n_cand]
    cand_token: np.ndarray    # int32 [n_cand]
    cand_parent: np.ndarray   # int32 [n_cand], -1 = root
    frontier: np.ndarray      # int32 [d, k]: candidates expanded after each level
    min_gap: float
    near_pairs: np.ndarray    # int32 [n_near, 2]: boundary pairs (before, after) with a gap below tau
    node_cand: np.ndarray     # int32 [n]: candidate index of each node (-1 for the root)

    def level_frontier(self, j: int, k: int, L: int):
        """The frontier after level j as a draft model needs it (Section 3.2, "Draft Tree Expansion": the k
        best tokens of a layer are expanded to the next one): per member p its token, the slot of its
        parent in the previous frontier (-1: the root), position id L + j + 1, its draft-node index
        1 + j k + p (the root is draft node 0) and the ancestor-or-self mask over draft nodes."""
        cands = [int(c) for c in self.frontier[j][:k]]
        tokens = np.array([self.cand_token[c] for c in cands], np.int32)
        prev = [int(c) for c in self.frontier[j - 1][:k]] if j > 0 else []
        parent_slot = np.array([prev.index(int(self.cand_parent[c])) if j > 0 else -1 for c in cands], np.int32)
        mask = np.zeros((k, 2), np.uint64)
        for p_, c in enumerate(cands):
            bits, cc, jj = 1, c, j                      # the root
            while True:
                slot = [int(x) for x in self.frontier[jj][:k]].index(cc)
                bits |= 1 << (1 + jj * k + slot)
                if jj == 0:
                    break
                cc, jj = int(self.cand_parent[cc]), jj - 1
            mask[p_] = (bits & 0xFFFFFFFFFFFFFFFF, bits >> 64)
        return dict(tokens=tokens, parent_slot=parent_slot, position_ids=np.full(k, L + j + 1, np.int32),
                    node_index=np.arange(1 + j * k, 1 + j * k + k, dtype=np.int32), mask=mask,
                    score=np.array([self.cand_score[c] for c in cands]))

    def node_rows(self, d: int, k: int, slots: int) -> np.ndarray:
        """int32 [n]: for every node the index level * slots + slot of the draft row its children were taken
        from (the root: row 0; a candidate that is the p-th member of the frontier after level j < d-1:
        row (j+1, p)), or -1 for a node that was not expanded."""
        row_of_cand = {}
        for j in range(d - 1):
            for p_, c in enumerate(self.frontier[j][:k]):
                row_of_cand[int(c)] = (j + 1) * slots + p_
        out = np.full(self.n_nodes, -1, np.int32)
        out[0] = 0
        for i in range(1, self.n_nodes):
            out[i] = row_of_cand.get(int(self.node_cand[i]), -1)
        return out


def tree_expand(root_token: int, logits: np.ndarray, TT: int, d: int, k: int, L: int,
                max_tt: int = 128, ret_stride: int | None = None, tau: float = 0.0,
                order_bias: np.ndarray | None = None) -> Tree:
    """Draft-tree construction. ``logits`` is fp32 [>=d][>=k][V]; level 0 uses slot 0.
    ``tau``: boundary pairs with a smaller score gap are listed in ``near_pairs``.
    ``order_bias`` (fp64 [n_cand]) is added where candidates are ordered (see the C++ header)."""
    logits = _c(logits, np.float32)
    assert logits.ndim == 3 and logits.shape[0] >= d and (d == 1 or logits.shape[1] >= k)
    V = logits.shape[2]
    ld_level = logits.shape[1] * V
    ld_row = V
    if ret_stride is None:
        ret_stride = d + 1
    n_cand = k + (d - 1) * k * k
    tokens = np.full(max_tt, -1, np.int32)
    parent = np.full(max_tt, -1, np.int32)
    depth = np.full(max_tt, -1, np.int32)
    pos = np.full(max_tt, -1, np.int32)
    mask = np.zeros((max_tt, 2), np.uint64)
    retrieve = np.full((max_tt, ret_stride), -1, np.int32)
    n_leaves = ctypes.c_int32()
    n_nodes = ctypes.c_int32()
    cand = np.zeros(n_cand, np.float64)
    ctok = np.zeros(n_cand, np.int32)
    cpar = np.zeros(n_cand, np.int32)
    frontier = np.zeros((d, k), np.int32)
    gap = ctypes.c_double()
    max_near = 64
    near = np.zeros((max_near, 2), np.int32)
    n_near = ctypes.c_int32()
    node_cand = np.full(max_tt, -1, np.int32)
    if order_bias is not None:
        order_bias = _c(order_bias, np.float64)
        assert order_bias.shape == (n_cand,)
    rc = _load().oracle_tree_expand(
        ctypes.c_int32(int(root_token)), _p(logits), ctypes.c_int64(ld_level), ctypes.c_int64(ld_row),
        V, TT, d, k, L, max_tt, ret_stride, _p(tokens), _p(parent), _p(depth), _p(pos), _p(mask),
        _p(retrieve), ctypes.byref(n_leaves), ctypes.byref(n_nodes), _p(cand), _p(ctok), _p(cpar),
        _p(frontier), ctypes.byref(gap), _p(order_bias) if order_bias is not None else None,
        ctypes.c_double(tau), _p(near), max_near, ctypes.byref(n_near), _p(node_cand))
    if rc != 0:
        raise ValueError(f"oracle_tree_expand rc={rc}")
    n = n_nodes.value
    return Tree(tokens[:n], parent[:n], depth[:n], pos[:n], mask[:n], retrieve[:n_leaves.value],
                n, n_leaves.value, cand, ctok, cpar, frontier, gap.value, near[:n_near.value].copy(),
                node_cand[:n].copy())


def tree_expand_swapped(root_token: int, logits: np.ndarray, TT: int, d: int, k: int, L: int,
                        tau: float, max_tt: int = 128, ret_stride: int | None = None):
    """The trees that differ from ``tree_expand``'s only by swaps among candidates whose scores
    lie within ``tau`` of each other at a selection boundary: for every non-empty subset of the
    near pairs, the tree built with the pair's second candidate ordered just before its first.
    Yields (flipped pairs, Tree).  At most 6 near pairs (63 variants) are explored."""
    base = tree_expand(root_token, logits, TT, d, k, L, max_tt, ret_stride, tau=tau)
    pairs = [tuple(int(x) for x in p) for p in base.near_pairs][:6]
    for subset in range(1, 1 << len(pairs)):
        bias = np.zeros(base.cand_score.shape[0], np.float64)
        flipped = []
        for i, (before, after) in enumerate(pairs):
            if subset >> i & 1:
                # lift `after` just above `before` (1e-9 is far above fp64 rounding of a score
                # and far below any tau worth the name)
                bias[after] += base.cand_score[before] - base.cand_score[after] + 1e-9
                flipped.append((before, after))
        yield flipped, tree_expand(root_token, logits, TT, d, k, L, max_tt, ret_stride, tau=tau,
                                   order_bias=bias)


def tree_attention(q: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray, L: int,
                   mask: np.ndarray, scale: float, want_lse: bool = False):
    """q: uint16(bf16 bits) [n][Hq][D]; caches uint16 [Hkv][cap][D]; mask uint64 [n][2].
    Returns fp64 [n][Hq][D] (and lse [n][Hq])."""
    q = _c(q, np.uint16)
    k_cache = _c(k_cache, np.uint16)
    v_cache = _c(v_cache, np.uint16)
    mask = _c(mask, np.uint64)
    n, Hq, D = q.shape
    Hkv, cap, D2 = k_cache.shape
    assert D2 == D and v_cache.shape == k_cache.shape and mask.shape == (n, 2)
    assert L + n <= cap
    out = np.empty((n, Hq, D), np.float64)
    lse = np.empty((n, Hq), np.float64) if want_lse else None
    rc = _load().oracle_tree_attention(
        n, Hq, Hkv, D, L, _p(q), _p(k_cache), _p(v_cache), ctypes.c_int64(cap * D),
        ctypes.c_int64(D), _p(mask), ctypes.c_double(scale), _p(out),
        _p(lse) if want_lse else None)
    if rc != 0:
        raise ValueError(f"oracle_tree_attention rc={rc}")
    return (out, lse) if want_lse else out


@dataclass
class Accept:
    target_argmax: np.ndarray  # int32 [n]
    path: np.ndarray           # int32 [a+1]
    accept_len: int
    out_tokens: np.ndarray     # int32 [a+1]


def verify_accept(target_logits: np.ndarray, tokens: np.ndarray, parent: np.ndarray,
                  path_cap: int = 17) -> Accept:
    target_logits = _c(target_logits, np.float32)
    tokens = _c(tokens, np.int32)
    parent = _c(parent, np.int32)
    n, V = target_logits.shape
    assert tokens.shape[0] >= n and parent.shape[0] >= n
    tgt = np.empty(n, np.int32)
    path = np.empty(path_cap, np.int32)
    out = np.empty(path_cap, np.int32)
    a = ctypes.c_int32()
    rc = _load().oracle_verify_accept(n, V, _p(target_logits), ctypes.c_int64(V), _p(tokens),
                                      _p(parent), path_cap, _p(tgt), _p(path), ctypes.byref(a),
                                      _p(out))
    if rc != 0:
        raise ValueError(f"oracle_verify_accept rc={rc}")
    return Accept(tgt, path[:a.value + 1].copy(), a.value, out[:a.value + 1].copy())


@dataclass
class SampledAccept:
    path: np.ndarray        # int32 [a+1]
    accept_len: int
    out_tokens: np.ndarray  # int32 [a+1]: the accepted draft tokens, then the drawn token
    min_margin: float


def verify_accept_sampled(target_logits: np.ndarray, draft_rows: np.ndarray, node_row: np.ndarray,
                          tokens: np.ndarray, parent: np.ndarray, temperature: float,
                          u_accept: np.ndarray, u_sample: np.ndarray, path_cap: int = 17) -> SampledAccept:
    """Acceptance under sampling.  target_logits fp32 [n][V]; draft_rows fp32 [R][V];
    node_row int32 [n]: the draft row a node's children were taken from (-1: none);
    u_accept fp64 [path_cap][max_children], u_sample fp64 [path_cap]: uniforms in (0, 1)."""
    target_logits = _c(target_logits, np.float32)
    draft_rows = _c(draft_rows, np.float32)
    node_row = _c(node_row, np.int32)
    tokens = _c(tokens, np.int32)
    parent = _c(parent, np.int32)
    u_accept = _c(u_accept, np.float64)
    u_sample = _c(u_sample, np.float64)
    n, V = target_logits.shape
    assert draft_rows.shape[1] == V and u_accept.shape[0] >= path_cap and u_sample.shape[0] >= path_cap
    path = np.empty(path_cap, np.int32)
    out = np.empty(path_cap, np.int32)
    a = ctypes.c_int32()
    margin = ctypes.c_double()
    rc = _load().oracle_verify_accept_sampled(
        n, V, _p(target_logits), ctypes.c_int64(V), _p(draft_rows), ctypes.c_int64(V), _p(node_row), _p(tokens),
        _p(parent), ctypes.c_double(temperature), _p(u_accept), int(u_accept.shape[1]), _p(u_sample), path_cap,
        _p(path), ctypes.byref(a), _p(out), ctypes.byref(margin))
    if rc != 0:
        raise ValueError(f"oracle_verify_accept_sampled rc={rc}")
    return SampledAccept(path[:a.value + 1].copy(), a.value, out[:a.value + 1].copy(), margin.value)


def kv_compact(k_cache: np.ndarray, v_cache: np.ndarray, L: int, path: np.ndarray) -> int:
    """In-place on the given uint16 [Hkv][cap][D] arrays (via an internal copy). Returns L'."""
    assert k_cache.dtype == np.uint16 and v_cache.dtype == np.uint16
    assert k_cache.flags.c_contiguous and v_cache.flags.c_contiguous
    Hkv, cap, D = k_cache.shape
    path = _c(path, np.int32)
    a = path.shape[0] - 1
    rc = _load().oracle_kv_compact(Hkv, D, L, _p(path), a, _p(k_cache), _p(v_cache),
                                   ctypes.c_int64(cap * D), ctypes.c_int64(D),
                                   ctypes.c_int64(k_cache.size))
    if rc != 0:
        raise ValueError(f"oracle_kv_compact rc={rc}")
    return L + a + 1


# ------------------------------------------------------------------------------ controller
@dataclass
class ControllerState:
    """Per-sequence state of the action cache (Algorithm 1)."""
    cache_step: int = 0        # position inside the cache interval; 0 = the policy is asked at the next step
    action: int = -1           # index of the cached action
    reward_sum: float = 0.0    # sum of accepted tokens / second over the steps of the open interval
    reward_steps: int = 0


def policy_logits(state_vec: np.ndarray, w1, b1, w2, b2, w3, b3) -> np.ndarray:
    """The policy network (Appendix A: two hidden layers of 128 units) in fp64 on the state
    s_t = concat(h, m, l) (Eq. 4): logits = W3 tanh(W2 tanh(W1 s + b1) + b2) + b3.  (tanh is the
    default activation of the Stable-Baselines3 policy the paper uses; the paper does not name it.)"""
    s = np.asarray(state_vec, np.float64)
    h1 = np.tanh(np.asarray(w1, np.float64) @ s + np.asarray(b1, np.float64))
    h2 = np.tanh(np.asarray(w2, np.float64) @ h1 + np.asarray(b2, np.float64))
    return np.asarray(w3, np.float64) @ h2 + np.asarray(b3, np.float64)


def controller_step(st: ControllerState, state_vec, weights, actions: np.ndarray, interval: int,
                    temperature: float, u: float, prev_accept_len, prev_elapsed_s):
    """One decoding step of Algorithm 1 (action caching) with the reward of Eq. 5.

    prev_accept_len / prev_elapsed_s describe the step that has just finished (None before the first
    step): its reward, tokens emitted (accepted drafts + 1) per second (Eq. 3), is added to the open
    interval.  When cache_step is 0 the interval is closed -- r_avg (Eq. 5), the mean of its rewards, is
    reported -- and the policy is asked: arg-max of its logits at temperature 0, else a draw from
    softmax(logits / temperature) by inverse CDF with u.  The chosen (TT, d, k) is then used for
    `interval` consecutive steps.  Returns (new state, (TT, d, k), r_avg or None, logits or None,
    margin): margin is the distance of the choice from flipping (top-2 logit gap, or the CDF distance)."""
    st = ControllerState(st.cache_step, st.action, st.reward_sum, st.reward_steps)
    if prev_accept_len is not None:
        st.reward_sum += (int(prev_accept_len) + 1) / float(prev_elapsed_s)
        st.reward_steps += 1
    r_avg, logits, margin = None, None, float("inf")
    if st.cache_step == 0 or st.action < 0:
        if st.reward_steps > 0:
            r_avg = st.reward_sum / st.reward_steps
        st.reward_sum, st.reward_steps = 0.0, 0
        logits = policy_logits(state_vec, *weights)
        if temperature <= 0.0:
            order = np.argsort(-logits, kind="stable")
            st.action = int(order[0])
            if len(order) > 1:
                margin = float(logits[order[0]] - logits[order[1]])
        else:
            z = logits / temperature
            p = np.exp(z - z.max())
            p /= p.sum()
            cdf = np.cumsum(p)
            target = u * cdf[-1]
            st.action = int(min(np.searchsorted(cdf, target, side="right"), len(p) - 1))
            lo = cdf[st.action - 1] if st.action > 0 else 0.0
            margin = float(min(target - lo, cdf[st.action] - target)) if st.action < len(p) - 1 else float(target - lo)
        st.cache_step = 1
    else:
        st.cache_step += 1
    if st.cache_step >= interval:
        st.cache_step = 0
    tt, d, k = (int(x) for x in actions[st.action])
    return st, (tt, d, k), r_avg, logits, margin
