"""Pins for the oracle's tree-masked attention (Section 3.2, Verification Phase: every tree
token is scored in one target pass, each seeing the prefix and its own ancestors)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_12212_b200 import synth


def bf16(x):
    x = np.asarray(x, np.float32)
    b = synth.to_bf16_bits(x.reshape(-1)).reshape(x.shape)
    return b if x.ndim else b[()]


def f64(b):
    return synth.bf16_bits_to_f32(b).astype(np.float64)


def chain_mask(n):
    m = np.zeros((n, 2), np.uint64)
    for i in range(n):
        v = (1 << (i + 1)) - 1
        m[i, 0] = v & 0xFFFFFFFFFFFFFFFF
        m[i, 1] = v >> 64
    return m


def make(rng, n, Hq, Hkv, D, L, cap=None):
    cap = cap or (L + n + 3)
    q = bf16(rng.normal(size=(n, Hq, D)))
    kc = bf16(rng.normal(size=(Hkv, cap, D)))
    vc = bf16(rng.normal(size=(Hkv, cap, D)))
    return q, kc, vc


@pytest.mark.parametrize("n,Hq,Hkv,D,L", [(9, 4, 1, 64, 37), (70, 6, 3, 32, 5), (5, 2, 2, 128, 0)])
def test_chain_tree_equals_causal_attention(n, Hq, Hkv, D, L):
    """A chain-shaped tree is ordinary causal attention over prefix + chain: compared with a
    separately written loop and with the library's scaled-dot-product attention."""
    rng = np.random.default_rng(n)
    q, kc, vc = make(rng, n, Hq, Hkv, D, L)
    scale = 1.0 / np.sqrt(D)
    out, lse = oracle.tree_attention(q, kc, vc, L, chain_mask(n), scale, want_lse=True)
    G = Hq // Hkv
    Q, K, Vv = f64(q), f64(kc), f64(vc)
    # (1) plain loop
    ref = np.zeros_like(out)
    for t in range(n):
        for h in range(Hq):
            keys = K[h // G, : L + t + 1]
            s = keys @ Q[t, h] * scale
            p = np.exp(s - s.max())
            ref[t, h] = (p[:, None] * Vv[h // G, : L + t + 1]).sum(0) / p.sum()
            assert lse[t, h] == pytest.approx(s.max() + np.log(p.sum()), abs=1e-10)
    np.testing.assert_allclose(out, ref, atol=1e-12)
    # (2) library routine, fp64, boolean mask, KV heads repeated for GQA
    tq = torch.from_numpy(Q).permute(1, 0, 2)[None]                       # [1,Hq,n,D]
    tk = torch.from_numpy(K[:, : L + n]).repeat_interleave(G, 0)[None]    # [1,Hq,L+n,D]
    tv = torch.from_numpy(Vv[:, : L + n]).repeat_interleave(G, 0)[None]
    allow = torch.zeros(n, L + n, dtype=torch.bool)
    for t in range(n):
        allow[t, : L + t + 1] = True
    lib = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=allow, scale=scale)
    np.testing.assert_allclose(out, lib[0].permute(1, 0, 2).numpy(), atol=1e-12)


def test_one_node_tree_is_plain_decode():
    rng = np.random.default_rng(0)
    n, Hq, Hkv, D, L = 1, 8, 2, 64, 200
    q, kc, vc = make(rng, n, Hq, Hkv, D, L)
    out = oracle.tree_attention(q, kc, vc, L, chain_mask(1), 0.125)
    Q, K, Vv = f64(q), f64(kc), f64(vc)
    for h in range(Hq):
        s = K[h // 4, : L + 1] @ Q[0, h] * 0.125
        p = np.exp(s - s.max())
        p /= p.sum()
        np.testing.assert_allclose(out[0, h], p @ Vv[h // 4, : L + 1], atol=1e-12)


def random_tree_mask(rng, n):
    parent = [-1] + [int(rng.integers(0, i)) for i in range(1, n)]
    m = np.zeros((n, 2), np.uint64)
    for i in range(n):
        v = 0
        c = i
        while c >= 0:
            v |= 1 << c
            c = parent[c]
        m[i, 0] = v & 0xFFFFFFFFFFFFFFFF
        m[i, 1] = v >> 64
    return parent, m


def test_closed_forms():
    rng = np.random.default_rng(3)
    n, Hq, Hkv, D, L = 100, 2, 1, 32, 19
    q, kc, vc = make(rng, n, Hq, Hkv, D, L)
    parent, mask = random_tree_mask(rng, n)
    # all-zero K: uniform weights => mean of the allowed V rows
    zk = np.zeros_like(kc)
    out = oracle.tree_attention(q, zk, vc, L, mask, 1.0)
    Vv = f64(vc)
    for t in (0, 1, 63, 64, 65, 99):
        anc = [j for j in range(n) if (int(mask[t, j >> 6]) >> (j & 63)) & 1]
        rows = list(range(L)) + [L + j for j in anc]
        np.testing.assert_allclose(out[t, 1], Vv[0, rows].mean(0), atol=1e-12)
    # one key dominating by a wide margin => output is its V row
    kc2 = np.zeros_like(kc)
    q2 = np.zeros_like(q)
    q2[:, :, 0] = bf16(np.float32(8.0))
    kc2[0, 4, 0] = bf16(np.float32(16.0))            # prefix slot 4: score 128 above the rest
    out = oracle.tree_attention(q2, kc2, vc, L, mask, 1.0)
    np.testing.assert_allclose(out[:, 0], np.broadcast_to(Vv[0, 4], (n, D)), atol=1e-30)


def test_prefix_permutation_invariance_and_poison_slots():
    rng = np.random.default_rng(4)
    n, Hq, Hkv, D, L = 40, 4, 2, 64, 50
    q, kc, vc = make(rng, n, Hq, Hkv, D, L, cap=L + n + 20)
    parent, mask = random_tree_mask(rng, n)
    base = oracle.tree_attention(q, kc, vc, L, mask, 0.125)
    # permuting the prefix slots changes nothing
    perm = rng.permutation(L)
    k2, v2 = kc.copy(), vc.copy()
    k2[:, :L] = kc[:, perm]
    v2[:, :L] = vc[:, perm]
    np.testing.assert_allclose(oracle.tree_attention(q, k2, v2, L, mask, 0.125), base, atol=1e-12)
    # huge values in slots past L+n never matter
    k3, v3 = kc.copy(), vc.copy()
    k3[:, L + n:] = bf16(np.float32(1e4))
    v3[:, L + n:] = bf16(np.float32(1e4))
    assert np.array_equal(oracle.tree_attention(q, k3, v3, L, mask, 0.125), base)
    # huge values at a non-ancestor tree slot do not reach a node
    leaf = n - 1
    anc = {j for j in range(n) if (int(mask[leaf, j >> 6]) >> (j & 63)) & 1}
    other = next(j for j in range(n) if j not in anc)
    k4, v4 = kc.copy(), vc.copy()
    k4[:, L + other] = bf16(np.float32(1e4))
    v4[:, L + other] = bf16(np.float32(1e4))
    out = oracle.tree_attention(q, k4, v4, L, mask, 0.125)
    assert np.array_equal(out[leaf], base[leaf])
    assert not np.array_equal(out[other], base[other])


def test_gqa_head_to_kv_head_mapping():
    """Query head h reads KV head h // (Hq/Hkv): make KV heads constant-valued and distinct."""
    n, Hq, Hkv, D, L = 3, 6, 3, 16, 4
    rng = np.random.default_rng(7)
    q, kc, vc = make(rng, n, Hq, Hkv, D, L)
    for g in range(Hkv):
        vc[g] = bf16(np.float32(g + 1))
    out = oracle.tree_attention(q, kc, vc, L, chain_mask(n), 0.25)
    for h in range(Hq):
        np.testing.assert_allclose(out[:, h], h // 2 + 1, atol=1e-12)


def test_lse_matches_library_logsumexp_and_the_closed_form():
    """The optional log-sum-exp output: against scipy's and torch's logsumexp over score rows
    built by one matrix product per KV head (not the oracle's per-key loop), and against the
    closed form log(#allowed keys) when every score is zero."""
    from scipy.special import logsumexp
    rng = np.random.default_rng(11)
    n, Hq, Hkv, D, L = 70, 6, 2, 64, 23
    q, kc, vc = make(rng, n, Hq, Hkv, D, L)
    parent, mask = random_tree_mask(rng, n)
    scale = 0.37
    _, lse = oracle.tree_attention(q, kc, vc, L, mask, scale, want_lse=True)
    G = Hq // Hkv
    Q, K = f64(q), f64(kc)
    allow = np.zeros((n, L + n), bool)
    allow[:, :L] = True
    for t in range(n):
        for j in range(n):
            allow[t, L + j] = (int(mask[t, j >> 6]) >> (j & 63)) & 1
    for g in range(Hkv):
        scores = np.einsum("thd,jd->thj", Q[:, g * G:(g + 1) * G], K[g, : L + n]) * scale   # [n][G][L+n]
        masked = np.where(allow[:, None, :], scores, -np.inf)
        np.testing.assert_allclose(lse[:, g * G:(g + 1) * G], logsumexp(masked, axis=-1), atol=1e-11)
        np.testing.assert_allclose(lse[:, g * G:(g + 1) * G],
                                   torch.logsumexp(torch.from_numpy(masked), dim=-1).numpy(), atol=1e-11)
    _, lse0 = oracle.tree_attention(q, np.zeros_like(kc), vc, L, mask, scale, want_lse=True)
    depth = np.array([bin((int(mask[t, 1]) << 64) | int(mask[t, 0])).count("1") for t in range(n)])
    np.testing.assert_allclose(lse0, np.log(L + depth)[:, None].repeat(Hq, 1), atol=1e-12)
