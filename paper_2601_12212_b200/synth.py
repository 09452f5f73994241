"""Seeded synthetic inputs for the speculative-step hot path.

Everything here is input generation: a counter-based random number generator,
the five workload descriptions, the per-step (TT, d, k) schedule, and the draft /
target logits and Q/K/V tensors with the stated distributions.  None of the
method's arithmetic (top-k, scoring, tree building, attention, acceptance,
compaction) lives in this module, so both the CUDA path's callers and the CPU
checker may use it without sharing any of the computation under test.

All generators run on the host in numpy and are pure functions of their integer
keys, so any consumer sees identical bits for identical keys.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Tuple, Union

import numpy as np

MAX_TT = 128
MAX_K = 32
MAX_D = 16

# The paper's action space (Appendix A, "Action Space in Implementation").
ACTION_TT = (32, 48, 64, 80, 96, 128)
ACTION_D = (3, 4, 5, 6, 7, 8)
ACTION_K = (8, 12, 16, 20, 32)

# The per-step grid the ragged / 13B-shaped workloads draw from.
GRID_TT = (16, 32, 48, 60, 80)
GRID_D = (3, 4, 5, 6, 7, 8)
GRID_K = tuple(range(4, 13))


def action_space(filtered: bool = False):
    """All (TT, d, k) of the paper's grid (6*6*5 = 180); ``filtered`` keeps TT <= k**(d-1)."""
    out = []
    for tt in ACTION_TT:
        for d in ACTION_D:
            for k in ACTION_K:
                if filtered and tt > k ** (d - 1):
                    continue
                out.append((tt, d, k))
    return out


# --------------------------------------------------------------------------- RNG
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_GOLD = np.uint64(0x9E3779B97F4A7C15)


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def stream_key(*ints: int) -> np.uint64:
    """Fold a tuple of integers (seed, config, step, sequence, layer, tensor id, ...) into a key."""
    with np.errstate(over="ignore"):
        h = np.array([0x243F6A8885A308D3], dtype=np.uint64)
        for v in ints:
            h = _mix(h + np.uint64(int(v) & 0xFFFFFFFFFFFFFFFF) * _GOLD + np.uint64(1))
        return h[0]


def bits(key: np.uint64, n: int, offset: int = 0) -> np.ndarray:
    """n 64-bit words: word i depends only on (key, offset + i)."""
    with np.errstate(over="ignore"):
        idx = np.arange(offset + 1, offset + n + 1, dtype=np.uint64)
        return _mix(np.uint64(key) + idx * _GOLD)


def uniform(key, n: int, offset: int = 0) -> np.ndarray:
    """Uniform in the open interval (0, 1), fp64."""
    return ((bits(key, n, offset) >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / (1 << 53))


def normal(key, n: int) -> np.ndarray:
    """Standard normal, fp64 (Box-Muller on two independent streams)."""
    u1 = uniform(stream_key(int(key), 1), n)
    u2 = uniform(stream_key(int(key), 2), n)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def gumbel(key, n: int) -> np.ndarray:
    return -np.log(-np.log(uniform(key, n)))


def randint(key, n: int, lo: int, hi: int) -> np.ndarray:
    """Integers uniform in [lo, hi)."""
    return (lo + np.floor(uniform(key, n) * (hi - lo))).astype(np.int64).clip(lo, hi - 1)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32/fp64 values to bf16 (round to nearest even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------- configs
Range = Union[int, Tuple[int, int]]


@dataclass(frozen=True)
class Workload:
    index: int
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    vocab: int
    n_layers: int          # layer count of the model the shape is taken from
    kv_capacity: int
    steps: int
    logit_model: str       # "normal2" or "gumbel_peaked"
    schedule: str          # "fixed" or "grid"
    tt: int
    d: int
    k: int
    prefix: Range          # fixed length, or (lo, hi) inclusive per sequence
    p_agree: Union[float, Tuple[float, float]]
    hold: int = 4          # steps each drawn (TT, d, k) is kept for (action persistence)
    seed: int = 0


WORKLOADS = {
    1: Workload(1, "tiny", 1, 4, 1, 64, 1024, 1, 2048, 32, "normal2", "fixed", 16, 4, 4, 128, 0.8),
    2: Workload(2, "llama-3.1-8b-shaped", 1, 32, 8, 128, 128256, 32, 4096, 200, "gumbel_peaked",
                "fixed", 60, 7, 10, 1024, 0.8),
    3: Workload(3, "vicuna-13b-shaped", 1, 40, 40, 128, 32000, 40, 8192, 500, "gumbel_peaked",
                "grid", 80, 8, 12, 2048, 0.8),
    4: Workload(4, "llama-3.3-70b-shaped", 1, 64, 8, 128, 128256, 80, 8192, 200, "gumbel_peaked",
                "fixed", 96, 8, 12, 4096, 0.8),
    5: Workload(5, "ragged-8b-shaped", 8, 32, 8, 128, 128256, 32, 12288, 300, "gumbel_peaked",
                "grid", 80, 8, 12, (1024, 8192), (0.5, 0.9)),
}

# tensor ids for stream keys
_T_SCHED, _T_PREFIX, _T_AGREE, _T_ROOT, _T_DRAFT, _T_DRAFT_PEAK, _T_TGT, _T_TGT_PICK, _T_Q, _T_K, \
    _T_V, _T_PK, _T_PV = range(13)


def step_params(w: Workload, step: int, seq: int) -> Tuple[int, int, int]:
    """(TT, d, k) for this step and sequence; grid draws are held for ``w.hold`` steps."""
    if w.schedule == "fixed":
        return w.tt, w.d, w.k
    draw = step // w.hold
    u = uniform(stream_key(w.seed, w.index, _T_SCHED, seq, draw), 3)
    tt = GRID_TT[min(int(u[0] * len(GRID_TT)), len(GRID_TT) - 1)]
    d = GRID_D[min(int(u[1] * len(GRID_D)), len(GRID_D) - 1)]
    k = GRID_K[min(int(u[2] * len(GRID_K)), len(GRID_K) - 1)]
    return tt, d, k


def initial_prefix(w: Workload, seq: int) -> int:
    if isinstance(w.prefix, tuple):
        lo, hi = w.prefix
        return int(randint(stream_key(w.seed, w.index, _T_PREFIX, seq), 1, lo, hi + 1)[0])
    return int(w.prefix)


def agreement_prob(w: Workload, seq: int) -> float:
    if isinstance(w.p_agree, tuple):
        lo, hi = w.p_agree
        return float(lo + (hi - lo) * uniform(stream_key(w.seed, w.index, _T_AGREE, seq), 1)[0])
    return float(w.p_agree)


def root_token(w: Workload, step: int, seq: int) -> int:
    return int(randint(stream_key(w.seed, w.index, _T_ROOT, seq, step), 1, 0, w.vocab)[0])


def _peaked_rows(g: np.ndarray, peak: np.ndarray, top1: float = 0.7) -> np.ndarray:
    """Given fp32 Gumbel noise rows, set row[peak] so that its softmax probability is ``top1``."""
    rows = g.astype(np.float32)
    r = np.arange(rows.shape[0])
    x = rows.astype(np.float64)
    x[r, peak] = -np.inf
    mx = x.max(axis=1)
    rest = mx + np.log(np.exp(x - mx[:, None]).sum(axis=1))
    rows[r, peak] = (rest + np.log(top1 / (1.0 - top1))).astype(np.float32)
    return rows


def draft_logits(w: Workload, step: int, seq: int, d: int, k: int) -> np.ndarray:
    """fp32 [d][k][V]: the draft model's output rows for each level's frontier slots.
    Level 0 only uses slot 0.  Row contents do not depend on (d, k) beyond the extent."""
    V = w.vocab
    out = np.empty((d, k, V), np.float32)
    for lvl in range(d):
        key = stream_key(w.seed, w.index, _T_DRAFT, seq, step, lvl)
        if w.logit_model == "normal2":
            out[lvl] = (2.0 * normal(key, k * V)).reshape(k, V).astype(np.float32)
        else:
            g = gumbel(key, k * V).reshape(k, V)
            peak = randint(stream_key(w.seed, w.index, _T_DRAFT_PEAK, seq, step, lvl), k, 0, V)
            out[lvl] = _peaked_rows(g, peak)
    return out


def target_logits(w: Workload, step: int, seq: int, tokens: np.ndarray, parent: np.ndarray,
                  n: int, p_agree: float) -> np.ndarray:
    """fp32 [n][V]: the target model's output after each tree node.  With probability
    ``p_agree`` (and if the node has a child in the tree) the strict maximum is the token of
    the node's first child, otherwise a token that none of its children carries."""
    V = w.vocab
    tokens = np.asarray(tokens[:n], dtype=np.int64)
    parent = np.asarray(parent[:n], dtype=np.int64)
    key = stream_key(w.seed, w.index, _T_TGT, seq, step)
    pick = uniform(stream_key(w.seed, w.index, _T_TGT_PICK, seq, step, 0), n)
    alt = randint(stream_key(w.seed, w.index, _T_TGT_PICK, seq, step, 1), n, 0, V)
    peak = np.empty(n, np.int64)
    for i in range(n):
        kids = np.nonzero(parent == i)[0]
        kid_tokens = set(int(t) for t in tokens[kids])
        if kids.size and pick[i] < p_agree:
            peak[i] = tokens[kids[0]]
        else:
            t = int(alt[i])
            while t in kid_tokens:
                t = (t + 1) % V
            peak[i] = t
    if w.logit_model == "normal2":
        rows = (2.0 * normal(key, n * V)).reshape(n, V).astype(np.float32)
        r = np.arange(n)
        rows[r, peak] = rows.max(axis=1) + np.float32(1.0)
        return rows
    return _peaked_rows(gumbel(key, n * V).reshape(n, V), peak)


def prefix_kv(w: Workload, seq: int, layer: int, length: int):
    """bf16 bit patterns, two arrays [Hkv][length][D]: the prefix K and V of one layer."""
    shape = (w.n_kv_heads, length, w.head_dim)
    kk = to_bf16_bits(normal(stream_key(w.seed, w.index, _T_PK, seq, layer), int(np.prod(shape))))
    vv = to_bf16_bits(normal(stream_key(w.seed, w.index, _T_PV, seq, layer), int(np.prod(shape))))
    return kk.reshape(shape), vv.reshape(shape)


def tree_kv(w: Workload, step: int, seq: int, layer: int, n: int):
    """bf16 bit patterns, two arrays [Hkv][n][D]: K and V of this step's n tree tokens."""
    shape = (w.n_kv_heads, n, w.head_dim)
    kk = to_bf16_bits(normal(stream_key(w.seed, w.index, _T_K, seq, step, layer), int(np.prod(shape))))
    vv = to_bf16_bits(normal(stream_key(w.seed, w.index, _T_V, seq, step, layer), int(np.prod(shape))))
    return kk.reshape(shape), vv.reshape(shape)


def queries(w: Workload, step: int, seq: int, layer: int, n: int) -> np.ndarray:
    """bf16 bit patterns [n][Hq][D]."""
    shape = (n, w.n_q_heads, w.head_dim)
    return to_bf16_bits(normal(stream_key(w.seed, w.index, _T_Q, seq, step, layer),
                               int(np.prod(shape)))).reshape(shape)
