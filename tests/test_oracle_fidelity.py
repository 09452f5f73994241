"""Whole-step pin: the paper's lossless-fidelity property (Section 3, "Lossless Output
Fidelity": greedy speculative sampling with target verification reproduces greedy
auto-regressive decoding).  A tiny random-weight transformer is decoded twice -- plainly,
and through the oracle's tree construction, tree attention, acceptance and cache compaction
with random per-step (TT, d, k) -- and the two token streams must be identical."""
import numpy as np
import pytest

import oracle
from paper_2601_12212_b200 import synth

DM, NL, HQ, HKV, HD, V, FF, CAP = 64, 2, 4, 1, 16, 1024, 128, 640


def make_weights(seed):
    rng = np.random.default_rng(seed)
    w = {"E": rng.normal(size=(V, DM)), "out": rng.normal(size=(DM, V)) / np.sqrt(DM) * 3}
    pos = np.arange(CAP)[:, None] / (10000 ** (np.arange(0, DM, 2)[None] / DM))
    w["P"] = np.concatenate([np.sin(pos), np.cos(pos)], axis=1)
    for l in range(NL):
        w[f"q{l}"] = rng.normal(size=(DM, HQ * HD)) / np.sqrt(DM) * 2
        w[f"k{l}"] = rng.normal(size=(DM, HKV * HD)) / np.sqrt(DM) * 2
        w[f"v{l}"] = rng.normal(size=(DM, HKV * HD)) / np.sqrt(DM)
        w[f"o{l}"] = rng.normal(size=(HQ * HD, DM)) / np.sqrt(HQ * HD)
        w[f"a{l}"] = rng.normal(size=(DM, FF)) / np.sqrt(DM)
        w[f"b{l}"] = rng.normal(size=(FF, DM)) / np.sqrt(FF)
    return w


def rms(x):
    return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + 1e-6)


def rows(x, w):
    """Row-by-row product so that a row's result does not depend on how many rows there are."""
    return np.stack([r @ w for r in x])


class Cache:
    def __init__(self):
        self.k = [np.zeros((HKV, CAP, HD), np.uint16) for _ in range(NL)]
        self.v = [np.zeros((HKV, CAP, HD), np.uint16) for _ in range(NL)]
        self.L = 0


def target_forward(w, cache, tokens, pos_ids, mask):
    """Target model over the n tree tokens; their K/V are written at slots L..L+n-1."""
    n, L = len(tokens), cache.L
    x = w["E"][tokens] + w["P"][pos_ids]
    for l in range(NL):
        h = rms(x)
        q = synth.to_bf16_bits(rows(h, w[f"q{l}"])).reshape(n, HQ, HD)
        kk = synth.to_bf16_bits(rows(h, w[f"k{l}"])).reshape(n, HKV, HD)
        vv = synth.to_bf16_bits(rows(h, w[f"v{l}"])).reshape(n, HKV, HD)
        cache.k[l][:, L:L + n] = kk.transpose(1, 0, 2)
        cache.v[l][:, L:L + n] = vv.transpose(1, 0, 2)
        o = oracle.tree_attention(q, cache.k[l], cache.v[l], L, mask, 1.0 / np.sqrt(HD))
        x = x + rows(o.reshape(n, HQ * HD), w[f"o{l}"])
        x = x + rows(np.maximum(rows(rms(x), w[f"a{l}"]), 0.0), w[f"b{l}"])
    return rows(rms(x), w["out"]).astype(np.float32)


def draft_row(w, seq, noise_key):
    """The draft model: a noised copy of the target, evaluated densely on the last 24 tokens."""
    seq = seq[-24:]
    n = len(seq)
    x = w["E"][seq] + w["P"][np.arange(n)]
    causal = np.tril(np.ones((n, n), bool))
    for l in range(NL):
        h = rms(x)
        q = (h @ w[f"q{l}"]).reshape(n, HQ, HD)
        kk = (h @ w[f"k{l}"]).reshape(n, HKV, HD)
        vv = (h @ w[f"v{l}"]).reshape(n, HKV, HD)
        s = np.einsum("thd,sd->hts", q, kk[:, 0]) / np.sqrt(HD)
        s = np.where(causal[None], s, -np.inf)
        p = np.exp(s - s.max(-1, keepdims=True))
        p /= p.sum(-1, keepdims=True)
        o = np.einsum("hts,sd->thd", p, vv[:, 0]).reshape(n, HQ * HD)
        x = x + o @ w[f"o{l}"]
        x = x + np.maximum(rms(x) @ w[f"a{l}"], 0.0) @ w[f"b{l}"]
    logits = rms(x[-1]) @ w["out"]
    return (logits + 0.7 * synth.normal(noise_key, V)).astype(np.float32)


ONE = np.array([[1, 0]], np.uint64)


def decode_plain(w, prompt, n_new):
    cache = Cache()
    out, tok = [], None
    for t in prompt:
        logits = target_forward(w, cache, np.array([t]), np.array([cache.L]), ONE)
        cache.L += 1
        tok = int(np.argmax(logits[0]))
    while len(out) < n_new:
        out.append(tok)
        logits = target_forward(w, cache, np.array([tok]), np.array([cache.L]), ONE)
        cache.L += 1
        tok = int(np.argmax(logits[0]))
    return out


def decode_speculative(w, prompt, n_new, seed):
    rng = np.random.default_rng(seed)
    cache = Cache()
    root = None
    for t in prompt:
        logits = target_forward(w, cache, np.array([t]), np.array([cache.L]), ONE)
        cache.L += 1
        root = int(np.argmax(logits[0]))
    out, context = [root], list(prompt) + [root]
    accepted = []
    step = 0
    while len(out) < n_new:
        TT, d, k = int(rng.integers(1, 25)), int(rng.integers(1, 6)), int(rng.integers(1, 5))
        L = cache.L
        logits = np.zeros((d, k, V), np.float32)
        logits[0, 0] = draft_row(w, context, synth.stream_key(seed, step, 0, 0))
        for j in range(1, d):
            part = oracle.tree_expand(root, logits[:j], 128, j, k, L)
            for p, c in enumerate(part.frontier[j - 1]):
                path = []
                while c >= 0:
                    path.append(int(part.cand_token[c]))
                    c = int(part.cand_parent[c])
                logits[j, p] = draft_row(w, context + path[::-1], synth.stream_key(seed, step, j, p))
        tree = oracle.tree_expand(root, logits, TT, d, k, L)
        tl = target_forward(w, cache, tree.tokens, tree.position_ids, tree.mask)
        acc = oracle.verify_accept(tl, tree.tokens, tree.parent)
        for l in range(NL):
            oracle.kv_compact(cache.k[l], cache.v[l], L, acc.path)
        cache.L = L + acc.accept_len + 1
        out.extend(int(t) for t in acc.out_tokens)
        context.extend(int(t) for t in acc.out_tokens)
        root = int(acc.out_tokens[-1])
        accepted.append(acc.accept_len)
        step += 1
    return out[:n_new], accepted


@pytest.mark.parametrize("seed", range(20))
def test_speculative_greedy_equals_autoregressive_greedy(seed):
    w = make_weights(seed)
    prompt = [int(t) for t in np.random.default_rng(seed + 500).integers(0, V, size=6)]
    n_new = 256
    plain = decode_plain(w, prompt, n_new)
    spec, accepted = decode_speculative(w, prompt, n_new, seed)
    assert spec == plain
    # the test is only meaningful if drafts are sometimes accepted and sometimes rejected
    assert max(accepted) >= 1 and min(accepted) == 0
