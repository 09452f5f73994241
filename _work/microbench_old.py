"""Per-entry-point timings of libresps on synthetic shapes (CUDA events, inputs larger than L2).

    python -m paper_2601_12212_b200.microbench attention [2 3 4 5 long]
    python -m paper_2601_12212_b200.microbench vocab     [2 3 4 5]

The numbers name the synthetic workload (synth.WORKLOADS) whose shape is used.  `attention` times
resps_tree_attention over distinct KV-cache layers; `vocab` times resps_tree_expand (row scan +
tree build) and resps_verify_accept (arg-max + accept walk) over a pool of distinct logit sets.
Values are random (timing only); parity is the business of tests/.
"""
from __future__ import annotations

import math
import random
import sys

import numpy as np
import torch

from . import binding


def _chain_mask(B: int, T: int) -> torch.Tensor:
    mk = np.zeros((B, T, 2), np.uint64)
    for i in range(T):
        v = (1 << (i + 1)) - 1
        mk[:, i, 0] = v & 0xFFFFFFFFFFFFFFFF
        mk[:, i, 1] = v >> 64
    return torch.from_numpy(mk.view(np.int64)).cuda()


def attention(name, B, Hq, Hkv, D, Ls, ns, cap, layers, reps=5):
    T = 128
    ctx = binding.Context(Hq, Hkv, D, 1000, max_batch=B, max_tt=T, max_k=4, max_depth=4)
    steps = torch.tensor([[ns[s], 1, 1, Ls[s]] for s in range(B)], dtype=torch.int32, device="cuda")
    nn = torch.tensor(ns, dtype=torch.int32, device="cuda")
    q = torch.randn(B, T, Hq, D, device="cuda").bfloat16()
    o = torch.zeros_like(q)
    ks = [torch.randn(B, Hkv, cap, D, device="cuda").bfloat16() for _ in range(layers)]
    vs = [torch.randn(B, Hkv, cap, D, device="cuda").bfloat16() for _ in range(layers)]
    mask = _chain_mask(B, T)
    scale = 1 / math.sqrt(D)

    def call(l):
        binding.resps_tree_attention(ctx, steps, nn, B, q, o, None, ks[l], vs[l], Hkv * cap * D, cap * D, D,
                                     cap, mask, scale)
    for l in range(layers):
        call(l)
    torch.cuda.synchronize()
    # one CUDA graph of all layers, replayed: launch overhead of the host does not enter the timing
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        call(0)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=stream):
            for l in range(layers):
                binding.resps_tree_attention(ctx, steps, nn, B, q, o, None, ks[l], vs[l], Hkv * cap * D, cap * D,
                                             D, cap, mask, scale, stream=stream)
        graph.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps):
            graph.replay()
        b.record(stream)
        torch.cuda.synchronize()
    us = a.elapsed_time(b) * 1e3 / (reps * layers)
    byts = sum(2 * (Ls[s] + ns[s]) * Hkv * D * 2 + 2 * ns[s] * Hq * D * 2 for s in range(B))
    flops = sum(4 * ns[s] * Hq * (Ls[s] + ns[s]) * D for s in range(B))
    print(f"{name:30s} {us:8.2f} us/call  {byts / us / 1e3:8.1f} GB/s  {flops / us / 1e6:8.1f} TFLOP/s  "
          f"bytes={byts / 1e6:.2f}MB status={ctx.status()}", flush=True)
    ctx.close()


def vocab(name, B, V, TT, d, k, pool=6, reps=10):
    ctx = binding.Context(32, 8, 128, V, max_batch=B, max_tt=TT, max_k=k, max_depth=d)
    i32 = dict(dtype=torch.int32, device="cuda")
    steps = torch.tensor([[TT, d, k, 1000]] * B, **i32)
    root = torch.zeros(B, **i32)
    drafts = [torch.randn(B, d, k, V, device="cuda") * 2 for _ in range(pool)]
    targets = [torch.randn(B, TT, V, device="cuda") * 2 for _ in range(pool)]
    tokens, parent, depth, pos = (torch.zeros(B, TT, **i32) for _ in range(4))
    mask = torch.zeros(B, TT, 2, dtype=torch.int64, device="cuda")
    retr = torch.zeros(B, TT, d + 1, **i32)
    nl, nn, alen = (torch.zeros(B, **i32) for _ in range(3))
    amax = torch.zeros(B, TT, **i32)
    path, otok = torch.zeros(B, d + 1, **i32), torch.zeros(B, d + 1, **i32)

    def expand(i):
        binding.resps_tree_expand(ctx, steps, B, drafts[i], d * k * V, k * V, V, d, k, root, tokens, parent,
                                  depth, pos, mask, retr, nl, nn)

    def verify(i):
        binding.resps_verify_accept(ctx, steps, nn, B, targets[i], TT * V, V, tokens, parent, amax, path, alen,
                                    otok)
    for fn, nm, byts in ((expand, "expand", (1 + (d - 1) * k) * V * 4 * B), (verify, "verify", TT * V * 4 * B)):
        for i in range(pool):
            fn(i)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            for i in range(pool):
                fn(i)
        b.record()
        torch.cuda.synchronize()
        us = a.elapsed_time(b) * 1e3 / (reps * pool)
        print(f"{name:30s} {nm:7s} {us:8.2f} us  {byts / us / 1e3:8.1f} GB/s  bytes={byts / 1e6:.1f}MB "
              f"status={ctx.status()}", flush=True)
    ctx.close()


def main(argv):
    what = argv[0] if argv else "attention"
    which = argv[1:] or ["2", "3", "4", "5"]
    if what == "attention":
        if "2" in which:
            attention("cfg2 32q/8kv L=1024 n=60", 1, 32, 8, 128, [1024], [60], 4096, 32)
        if "3" in which:
            attention("cfg3 40q/40kv L=2048 n=48", 1, 40, 40, 128, [2048], [48], 8192, 8)
        if "4" in which:
            attention("cfg4 64q/8kv L=4096 n=96", 1, 64, 8, 128, [4096], [96], 8192, 40)
        if "5" in which:
            random.seed(0)
            Ls = [random.randint(1024, 8192) for _ in range(8)]
            ns = [random.choice([16, 32, 37, 48, 53, 60, 69, 80]) for _ in range(8)]
            attention("cfg5 ragged x8 32q/8kv", 8, 32, 8, 128, Ls, ns, 12288, 4)
        if "long" in which:  # not one of the workloads: the HBM-bound shape of workload 3 at a long context
            attention("MHA 40 heads L=32768 n=48", 1, 40, 40, 128, [32768], [48], 32768 + 128, 2)
            attention("32q/8kv L=65536 n=28", 1, 32, 8, 128, [65536], [28], 65536 + 128, 2)
    elif what == "vocab":
        if "2" in which:
            vocab("cfg2 V=128256 60/7/10", 1, 128256, 60, 7, 10)
        if "3" in which:
            vocab("cfg3 V=32000 80/8/12", 1, 32000, 80, 8, 12)
        if "4" in which:
            vocab("cfg4 V=128256 96/8/12", 1, 128256, 96, 8, 12)
        if "5" in which:
            vocab("cfg5 B=8 V=128256 80/8/12", 8, 128256, 80, 8, 12, pool=2)
    else:
        raise SystemExit(__doc__)


if __name__ == "__main__":
    main(sys.argv[1:])
