"""Pins for the oracle's draft-tree construction (Section 3.2, Draft Tree Expansion and
Confidence-Based Candidate Reranking; Algorithm 2, tree-building loop)."""
import json
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def log_softmax64(row):
    x = row.astype(np.float64)
    m = x.max()
    return x - (m + math.log(np.exp(x - m).sum()))


# ------------------------------------------------------------------ worked example
def test_hand_worked_example():
    g = json.load(open(os.path.join(GOLDEN, "tree_worked_example.json")))
    V, k, d = g["V"], g["k"], g["d"]
    logits = np.zeros((d, k, V), np.float32)
    logits[0, 0] = np.log(g["probs_level0_slot0"])
    logits[1, 0] = np.log(g["probs_level1_slot0"])
    logits[1, 1] = np.log(g["probs_level1_slot1"])
    for case in g["cases"]:
        t = oracle.tree_expand(g["root_token"], logits, case["TT"], d, k, g["L"])
        assert t.tokens.tolist() == case["tokens"]
        assert t.parent.tolist() == case["parent"]
        assert t.depth.tolist() == case["depth"]
        assert t.position_ids.tolist() == case["position_ids"]
        assert t.mask[:, 0].tolist() == case["mask_lo"] and not t.mask[:, 1].any()
        assert t.retrieve.tolist() == case["retrieve"]
        assert t.cand_token.tolist() == g["candidates"]["token"]
        assert t.cand_parent.tolist() == g["candidates"]["parent"]
        np.testing.assert_allclose(np.exp(t.cand_score), g["candidates"]["V_i"], rtol=1e-6)
        assert t.frontier[1].tolist() == g["frontier_after_level1"]
        if case["TT"] in (4,):
            assert t.min_gap == pytest.approx(math.log(0.275 / 0.27), abs=1e-6)


def test_near_pairs_and_swapped_trees_by_hand():
    """Near-tie support of the oracle, on values worked by hand from Section 3.2's V_i (product of
    the draft confidences along the root path).  k = 2, d = 3, V = 4.
      level 0, p = [.5, .4, .06, .04]:  c0 = tok 0 (V .5), c1 = tok 1 (V .4)
      level 1, after c0 p = [.6, .2, .15, .05]: c2 = tok 0 (.30), c3 = tok 1 (.10)
               after c1 p = [.05, .7499, .1501, .05]: c4 = tok 1 (.29996), c5 = tok 2 (.06004)
        frontier = [c2, c4], third is c3: the pair (c2, c4) is log(.30/.29996) = 1.3e-4 apart
      level 2, slot 0 p = [.1, .2, .3, .4]: c6 = tok 3, c7 = tok 2 under frontier[0]
               slot 1 p = [.9, .05, .03, .02]: c8 = tok 0, c9 = tok 1 under frontier[1]
    TT = 7 keeps the six best: c0, c1, c2, c4, c8 (.269964), c6 (.12); next is c3 (.10).
    With the pair swapped the slots change hands: c6 hangs under c4 and c8 under c2; the kept set
    stays (c8 = .27, c6 = .119984)."""
    logits = np.zeros((3, 2, 4), np.float32)
    logits[0, 0] = np.log([.5, .4, .06, .04])
    logits[1, 0] = np.log([.6, .2, .15, .05])
    logits[1, 1] = np.log([.05, .7499, .1501, .05])
    logits[2, 0] = np.log([.1, .2, .3, .4])
    logits[2, 1] = np.log([.9, .05, .03, .02])
    t = oracle.tree_expand(9, logits, 7, 3, 2, 0, tau=1e-3)
    assert t.tokens.tolist() == [9, 0, 1, 0, 1, 3, 0]
    assert t.parent.tolist() == [-1, 0, 0, 1, 2, 3, 4]
    assert t.min_gap == pytest.approx(math.log(.30 / .29996), abs=1e-6)
    assert t.near_pairs.tolist() == [[2, 4]]
    # a tau below the gap lists nothing, and then there is no swapped tree either
    assert oracle.tree_expand(9, logits, 7, 3, 2, 0, tau=1e-4).near_pairs.shape[0] == 0
    assert list(oracle.tree_expand_swapped(9, logits, 7, 3, 2, 0, tau=1e-4)) == []
    variants = list(oracle.tree_expand_swapped(9, logits, 7, 3, 2, 0, tau=1e-3))
    assert len(variants) == 1
    flipped, tv = variants[0]
    assert flipped == [(2, 4)]
    assert tv.tokens.tolist() == [9, 0, 1, 0, 1, 3, 0]
    assert tv.parent.tolist() == [-1, 0, 0, 1, 2, 4, 3]
    assert tv.frontier[1].tolist() == [4, 2]
    np.testing.assert_allclose(np.exp(tv.cand_score[[6, 8]]), [.119984, .27], rtol=1e-6)
    check_invariants(tv, logits, 9, 7, 3, 2, 0)
    # the last level's frontier is expanded by nobody: its order is no boundary (d = 2 here)
    t2 = oracle.tree_expand(9, logits, 100, 2, 2, 0, tau=1e-3)
    assert t2.near_pairs.shape[0] == 0 and t2.min_gap == float("inf")
    # the rerank boundary is one: TT = 4 keeps c0, c1, c2 and drops c4 by the same 1.3e-4
    t3 = oracle.tree_expand(9, logits, 4, 2, 2, 0, tau=1e-3)
    assert t3.near_pairs.tolist() == [[2, 4]] and t3.tokens.tolist() == [9, 0, 1, 0]
    (fl, tv3), = oracle.tree_expand_swapped(9, logits, 4, 2, 2, 0, tau=1e-3)
    assert tv3.tokens.tolist() == [9, 0, 1, 1] and tv3.parent.tolist() == [-1, 0, 0, 2]


# ---------------------------------------------------------------------- invariants
def check_invariants(t, logits, root, TT, d, k, L):
    n = t.n_nodes
    n_cand = k + (d - 1) * k * k
    assert n == min(TT, 1 + n_cand)
    assert t.tokens[0] == root and t.parent[0] == -1 and t.depth[0] == 0
    for i in range(1, n):
        p = int(t.parent[i])
        assert 0 <= p < i
        assert t.depth[i] == t.depth[p] + 1
        m = (int(t.mask[i, 1]) << 64) | int(t.mask[i, 0])
        mp = (int(t.mask[p, 1]) << 64) | int(t.mask[p, 0])
        assert m == mp | (1 << i)
        assert bin(m).count("1") == t.depth[i] + 1
    assert np.array_equal(t.position_ids, L + t.depth)
    # scores non-increasing along root paths (products of probabilities)
    for c in range(n_cand):
        if t.cand_parent[c] >= 0:
            assert t.cand_score[c] <= t.cand_score[t.cand_parent[c]]
        assert t.cand_score[c] <= 0.0
    # kept set: best m by score, ancestor closed
    order = sorted(range(n_cand), key=lambda c: (-t.cand_score[c], c))
    kept = sorted(order[: n - 1])
    assert [int(x) for x in t.cand_token[kept]] == t.tokens[1:].tolist()
    kept_set = set(kept)
    for c in kept:
        assert t.cand_parent[c] == -1 or int(t.cand_parent[c]) in kept_set
    if n - 1 < n_cand:
        worst_kept = min(t.cand_score[c] for c in kept) if kept else math.inf
        assert all(t.cand_score[c] <= worst_kept for c in range(n_cand) if c not in kept_set)
    # children of one parent carry distinct tokens
    for i in range(n):
        kids = [int(t.tokens[c]) for c in range(n) if t.parent[c] == i]
        assert len(kids) == len(set(kids))
    # retrieve rows: parent chains root -> leaf, ascending leaf index, cover all nodes
    leaves = [i for i in range(n) if not any(t.parent[c] == i for c in range(n))]
    assert t.n_leaves == len(leaves) and t.retrieve.shape[0] == len(leaves)
    covered = set()
    for row, leaf in zip(t.retrieve, leaves):
        path = [int(x) for x in row if x >= 0]
        assert path[0] == 0 and path[-1] == leaf
        assert all(x == -1 for x in row[len(path):])
        for a, b in zip(path[:-1], path[1:]):
            assert t.parent[b] == a
        covered.update(path)
    assert covered == set(range(n))


@pytest.mark.parametrize("seed", range(30))
def test_invariants_on_random_trees(seed):
    rng = np.random.default_rng(seed)
    V = int(rng.integers(16, 400))
    k = int(rng.integers(1, min(12, V) + 1))
    d = int(rng.integers(1, 9))
    TT = int(rng.integers(1, 129))
    L = int(rng.integers(0, 5000))
    logits = (rng.normal(size=(d, k, V)) * 3).astype(np.float32)
    root = int(rng.integers(0, V))
    t = oracle.tree_expand(root, logits, TT, d, k, L)
    check_invariants(t, logits, root, TT, d, k, L)


def test_tt_equal_to_pool_keeps_everything_and_larger_tt_clamps():
    rng = np.random.default_rng(5)
    V, k, d = 50, 3, 3
    logits = rng.normal(size=(d, k, V)).astype(np.float32)
    n_cand = k + (d - 1) * k * k
    a = oracle.tree_expand(1, logits, 1 + n_cand, d, k, 0)
    b = oracle.tree_expand(1, logits, 128, d, k, 0)
    assert a.n_nodes == b.n_nodes == 1 + n_cand
    assert a.tokens.tolist() == b.tokens.tolist() and a.parent.tolist() == b.parent.tolist()
    assert a.tokens[1:].tolist() == a.cand_token.tolist()
    one = oracle.tree_expand(1, logits, 1, d, k, 3)
    assert one.n_nodes == 1 and one.retrieve.tolist() == [[0, -1, -1, -1]]
    assert one.mask.tolist() == [[1, 0]]


# ------------------------------------------------------------------ special cases
@pytest.mark.parametrize("TT", [2, 4, 6, 40])
def test_k1_is_greedy_chain(TT):
    """k = 1: each level keeps the single most likely token => classic chain drafting
    (Section 3.2, Draft Phase), truncated by TT."""
    rng = np.random.default_rng(TT)
    V, d = 97, 5
    logits = rng.normal(size=(d, 1, V)).astype(np.float32)
    t = oracle.tree_expand(3, logits, TT, d, 1, 11)
    n = min(d, TT - 1) + 1
    assert t.n_nodes == n
    assert t.tokens[1:].tolist() == [int(np.argmax(logits[j, 0])) for j in range(n - 1)]
    assert t.parent.tolist() == [-1] + list(range(n - 1))
    assert t.retrieve.shape[0] == 1
    assert [x for x in t.retrieve[0] if x >= 0] == list(range(n))
    cum = np.cumsum([log_softmax64(logits[j, 0]).max() for j in range(d)])
    np.testing.assert_allclose(t.cand_score, cum, atol=1e-12)


@pytest.mark.parametrize("TT", [1, 3, 6, 50])
def test_d1_is_star_of_root_topk(TT):
    rng = np.random.default_rng(TT)
    V, k = 64, 5
    logits = rng.normal(size=(1, 1, V)).astype(np.float32)
    t = oracle.tree_expand(0, logits, TT, 1, k, 0)
    m = min(k, TT - 1)
    order = sorted(range(V), key=lambda i: (-float(logits[0, 0, i]), i))
    assert t.tokens[1:].tolist() == order[:m]
    assert (t.parent[1:] == 0).all() and (t.depth[1:] == 1).all()


# ---------------------------------------------------------------------- brute force
def brute_force_tree(root, logits, TT, d, k):
    """Independent restatement: nodes are root paths (tuples of child ranks chosen at
    each level); a path's value is the product of softmax probabilities along it.  Every
    path the expansion rule allows is enumerated, then all are ranked."""
    V = logits.shape[2]
    prob = lambda lvl, slot: np.exp(log_softmax64(logits[lvl, slot]))
    best = lambda p: sorted(range(V), key=lambda v: (-float(p[v]), v))[:k]

    # expanded[path] = (value, token, creation order); frontier = list of paths in slot order
    expanded = {}
    order = 0
    p0 = prob(0, 0)
    frontier = []
    for tok in best(p0):
        path = (tok,)
        expanded[path] = (math.log(p0[tok]), order)
        order += 1
        frontier.append(path)
    for lvl in range(1, d):
        layer = []
        for slot, par in enumerate(frontier):
            p = prob(lvl, slot)
            for tok in best(p):
                path = par + (tok,)
                expanded[path] = (expanded[par][0] + math.log(p[tok]), order)
                order += 1
                layer.append(path)
        layer.sort(key=lambda q: (-expanded[q][0], expanded[q][1]))
        frontier = layer[:k]
    ranked = sorted(expanded, key=lambda q: (-expanded[q][0], expanded[q][1]))
    kept = sorted(ranked[: max(0, TT - 1)], key=lambda q: expanded[q][1])
    nodes = [()] + kept
    idx = {q: i for i, q in enumerate(nodes)}
    tokens = [root] + [q[-1] for q in kept]
    parent = [-1] + [idx[q[:-1]] for q in kept]
    return tokens, parent


@pytest.mark.parametrize("seed", range(60))
def test_brute_force_enumeration_on_tiny_inputs(seed):
    rng = np.random.default_rng(1000 + seed)
    V = int(rng.integers(2, 7))
    k = int(rng.integers(1, min(2, V) + 1))
    d = int(rng.integers(1, 4))
    TT = int(rng.integers(1, 12))
    logits = rng.normal(size=(d, k, V)).astype(np.float32)
    if seed % 3 == 0:  # quantised logits: ties in value and in score
        logits = np.round(logits)
    t = oracle.tree_expand(7, logits, TT, d, k, 0)
    tokens, parent = brute_force_tree(7, logits, TT, d, k)
    if t.min_gap > 1e-9 or seed % 3:
        assert t.tokens.tolist() == tokens and t.parent.tolist() == parent
    else:  # exact score ties under rounding differences: only sizes are comparable
        assert t.n_nodes == len(tokens)


def test_level_frontier_of_the_worked_example():
    """The per-level view of the hand-worked example: after level 0 the frontier is candidates 0 and 1
    (tokens 0 and 1, children of the root, draft nodes 1 and 2); after level 1 it is candidates 2 (token 2
    under candidate 0) and 4 (token 3 under candidate 1): draft nodes 3 and 4 with masks root|1|3 and root|2|4."""
    g = json.load(open(os.path.join(GOLDEN, "tree_worked_example.json")))
    logits = np.zeros((2, 2, 4), np.float32)
    logits[0, 0] = np.log(g["probs_level0_slot0"])
    logits[1, 0] = np.log(g["probs_level1_slot0"])
    logits[1, 1] = np.log(g["probs_level1_slot1"])
    t = oracle.tree_expand(9, logits, 5, 2, 2, 7)
    f0 = t.level_frontier(0, 2, 7)
    assert f0["tokens"].tolist() == [0, 1] and f0["parent_slot"].tolist() == [-1, -1]
    assert f0["position_ids"].tolist() == [8, 8] and f0["node_index"].tolist() == [1, 2]
    assert f0["mask"][:, 0].tolist() == [0b011, 0b101]
    f1 = t.level_frontier(1, 2, 7)
    assert f1["tokens"].tolist() == [2, 3] and f1["parent_slot"].tolist() == [0, 1]
    assert f1["position_ids"].tolist() == [9, 9] and f1["node_index"].tolist() == [3, 4]
    assert f1["mask"][:, 0].tolist() == [0b01011, 0b10101]
    np.testing.assert_allclose(np.exp(f1["score"]), [0.275, 0.27], rtol=1e-6)
