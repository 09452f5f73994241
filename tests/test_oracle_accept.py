"""Pins for greedy verification / acceptance (Section 3.1 greedy rule; Section 3.2 Acceptance
Criterion at temperature 0) and KV-cache compaction (Appendix D, input update)."""
import numpy as np
import pytest

import oracle


def random_tree(rng, n, V, branching=3):
    tokens = [int(rng.integers(0, V))]
    parent = [-1]
    for i in range(1, n):
        while True:
            p = int(rng.integers(max(0, i - 6), i))
            t = int(rng.integers(0, V))
            sibs = [tokens[c] for c in range(i) if parent[c] == p]
            if t not in sibs and len(sibs) < branching:
                break
        tokens.append(t)
        parent.append(p)
    return np.array(tokens, np.int32), np.array(parent, np.int32)


def retrieve_rows(parent):
    n = len(parent)
    rows = []
    for i in range(n):
        if not any(parent[c] == i for c in range(n)):
            path = []
            c = i
            while c >= 0:
                path.append(c)
                c = int(parent[c])
            rows.append(path[::-1])
    return rows


def logits_with_argmax(rng, n, V, arg):
    x = rng.normal(size=(n, V)).astype(np.float32)
    x[np.arange(n), arg] = x.max(axis=1) + 1
    return x


@pytest.mark.parametrize("seed", range(25))
def test_accept_is_longest_matching_root_path(seed):
    rng = np.random.default_rng(seed)
    n, V = int(rng.integers(1, 60)), 12
    tokens, parent = random_tree(rng, n, V)
    tgt = rng.integers(0, V, size=n)
    # make agreement likely: with prob .7 point a node's target at one of its children
    for i in range(n):
        kids = [c for c in range(n) if parent[c] == i]
        if kids and rng.random() < 0.7:
            tgt[i] = tokens[kids[int(rng.integers(0, len(kids)))]]
    acc = oracle.verify_accept(logits_with_argmax(rng, n, V, tgt), tokens, parent)
    assert acc.target_argmax.tolist() == tgt.tolist()
    # brute force over the candidate paths
    best, best_row = -1, None
    for row in retrieve_rows(parent):
        m = 0
        while m + 1 < len(row) and tokens[row[m + 1]] == tgt[row[m]]:
            m += 1
        if m > best:
            best, best_row = m, row
    assert acc.accept_len == best
    assert acc.path.tolist() == best_row[: best + 1]
    path = acc.path.tolist()
    assert path[0] == 0 and all(parent[b] == a for a, b in zip(path[:-1], path[1:]))
    assert all(tokens[b] == tgt[a] for a, b in zip(path[:-1], path[1:]))
    assert acc.out_tokens.tolist() == [int(tokens[c]) for c in path[1:]] + [int(tgt[path[-1]])]
    # maximal: no child of the last node carries the target's token
    assert not any(parent[c] == path[-1] and tokens[c] == tgt[path[-1]] for c in range(n))


def test_chain_is_longest_common_prefix():
    """k = 1: accepted length = number of leading draft tokens equal to the target's greedy
    continuation (classic draft-then-verify, Section 3.2)."""
    rng = np.random.default_rng(0)
    V, n = 30, 9
    for agree in range(n):
        tokens = rng.integers(0, V, size=n).astype(np.int32)
        parent = np.arange(-1, n - 1).astype(np.int32)
        tgt = np.empty(n, np.int64)
        for i in range(n):
            nxt = tokens[i + 1] if i + 1 < n else 0
            tgt[i] = nxt if i < agree else (nxt + 1) % V
        acc = oracle.verify_accept(logits_with_argmax(rng, n, V, tgt), tokens, parent)
        assert acc.accept_len == min(agree, n - 1)
        assert acc.path.tolist() == list(range(acc.accept_len + 1))
        assert acc.out_tokens[-1] == tgt[acc.accept_len]


def test_full_and_zero_agreement():
    rng = np.random.default_rng(1)
    n, V = 40, 50
    tokens, parent = random_tree(rng, n, V)
    first_kid = {i: next((c for c in range(n) if parent[c] == i), None) for i in range(n)}
    tgt = np.array([tokens[first_kid[i]] if first_kid[i] is not None else 0 for i in range(n)])
    acc = oracle.verify_accept(logits_with_argmax(rng, n, V, tgt), tokens, parent)
    # follows first children down to a leaf
    cur, depth = 0, 0
    while first_kid[cur] is not None:
        cur, depth = first_kid[cur], depth + 1
    assert acc.accept_len == depth and acc.path[-1] == cur
    # zero agreement: a token no child carries
    tgt0 = np.array([next(t for t in range(V) if t not in
                          [tokens[c] for c in range(n) if parent[c] == i]) for i in range(n)])
    acc = oracle.verify_accept(logits_with_argmax(rng, n, V, tgt0), tokens, parent)
    assert acc.accept_len == 0 and acc.path.tolist() == [0] and acc.out_tokens.tolist() == [tgt0[0]]


def test_argmax_ties_take_lowest_id():
    x = np.zeros((2, 10), np.float32)
    x[0, [3, 7]] = 5
    x[1, :] = -1
    acc = oracle.verify_accept(x, np.array([0, 1], np.int32), np.array([-1, 0], np.int32))
    assert acc.target_argmax.tolist() == [3, 0]


@pytest.mark.parametrize("seed", range(6))
def test_compaction_is_a_gather(seed):
    rng = np.random.default_rng(seed)
    Hkv, cap, D, L = 3, 64, 8, int(rng.integers(0, 20))
    kc = rng.integers(0, 65535, size=(Hkv, cap, D)).astype(np.uint16)
    vc = rng.integers(0, 65535, size=(Hkv, cap, D)).astype(np.uint16)
    a = int(rng.integers(0, 9))
    path = np.concatenate([[0], np.sort(rng.choice(np.arange(1, 30), size=a, replace=False))])
    k0, v0 = kc.copy(), vc.copy()
    L2 = oracle.kv_compact(kc, vc, L, path)
    assert L2 == L + a + 1
    for j, p in enumerate(path):
        assert np.array_equal(kc[:, L + j], k0[:, L + p]) and np.array_equal(vc[:, L + j], v0[:, L + p])
    assert np.array_equal(kc[:, :L], k0[:, :L]) and np.array_equal(vc[:, :L], v0[:, :L])
    untouched = [s for s in range(L + a + 1, cap)]
    assert np.array_equal(kc[:, untouched], k0[:, untouched])


def test_compaction_identity_path_is_noop():
    rng = np.random.default_rng(9)
    kc = rng.integers(0, 65535, size=(2, 32, 4)).astype(np.uint16)
    vc = rng.integers(0, 65535, size=(2, 32, 4)).astype(np.uint16)
    k0, v0 = kc.copy(), vc.copy()
    oracle.kv_compact(kc, vc, 5, np.arange(6))
    assert np.array_equal(kc, k0) and np.array_equal(vc, v0)
