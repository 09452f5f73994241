#!/usr/bin/env python
"""Benchmark of the speculative-step hot path (expand + attention over all layers + verify +
compaction) on seeded synthetic inputs shaped like the paper's target models.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference]

Prints ONE JSON line.  `value` is microseconds per speculative step with all inputs resident
in HBM, measured with CUDA events around K replays of a captured CUDA graph of the step;
`e2e` is the same step driven from pinned HOST buffers (inputs copied in, results copied out
inside the timed region); `roofline` describes the dominant kernel (tree attention) from a
live CUDA-event measurement; `cpu_baseline` is the CPU oracle timed on this machine's host cores.
`--impl reference` times the CPU oracle alone.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2601_12212_b200 import synth  # noqa: E402

METRIC = "us_per_speculative_step"
UNIT = "us/step"
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes of one tree_attention_kernel launch on the benchmarked workload, from the ncu capture
# summarised in profiles/tree_attention_cfg2_ncu.md (set to None when the kernel changes).
ATTENTION_TRAFFIC_BYTES = 5018624


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return float(j["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------- reference (oracle) arm
def oracle_step_seconds(w: synth.Workload, attn_layers: int, step: int = 0):
    """One speculative step of the CPU oracle, with `attn_layers` of the workload's layers
    computed; returns per-phase seconds.  Single-threaded C++ (see oracle/)."""
    import oracle
    tt, d, k = synth.step_params(w, step, 0)
    L = synth.initial_prefix(w, 0)
    cap = L + tt + 8
    dl = synth.draft_logits(w, step, 0, d, k)
    t0 = time.perf_counter()
    tree = oracle.tree_expand(synth.root_token(w, step, 0), dl, tt, d, k, L)
    t_expand = time.perf_counter() - t0
    n = tree.n_nodes
    tl = synth.target_logits(w, step, 0, tree.tokens, tree.parent, n, synth.agreement_prob(w, 0))
    t_attn = 0.0
    caches = []
    for l in range(attn_layers):
        kc = np.zeros((w.n_kv_heads, cap, w.head_dim), np.uint16)
        vc = np.zeros_like(kc)
        pk, pv = synth.prefix_kv(w, 0, l, L)
        tk, tv = synth.tree_kv(w, step, 0, l, n)
        kc[:, :L], vc[:, :L] = pk, pv
        kc[:, L:L + n], vc[:, L:L + n] = tk, tv
        q = synth.queries(w, step, 0, l, n)
        t0 = time.perf_counter()
        oracle.tree_attention(q, kc, vc, L, tree.mask, 1.0 / np.sqrt(w.head_dim))
        t_attn += time.perf_counter() - t0
        caches.append((kc, vc))
    t0 = time.perf_counter()
    acc = oracle.verify_accept(tl, tree.tokens, tree.parent)
    t_verify = time.perf_counter() - t0
    t0 = time.perf_counter()
    for kc, vc in caches:
        oracle.kv_compact(kc, vc, L, acc.path)
    t_compact = time.perf_counter() - t0
    return {"expand": t_expand, "attn_per_layer": t_attn / max(1, attn_layers), "verify": t_verify,
            "compact_per_layer": t_compact / max(1, attn_layers), "n_nodes": n}


def oracle_us_per_step(w, parts):
    return 1e6 * (parts["expand"] + parts["verify"] +
                  w.n_layers * (parts["attn_per_layer"] + parts["compact_per_layer"]))


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    layers = 2
    for i in range(args.warmup):
        oracle_step_seconds(w, 1, step=i)
    t0 = time.perf_counter()
    vals = [oracle_us_per_step(w, oracle_step_seconds(w, layers, step=i)) for i in range(args.steps)]
    wall = time.perf_counter() - t0
    v = float(np.mean(vals))
    sample = (f"per step: tree construction + verification of one full step and {layers} of the "
              f"{w.n_layers} layers' attention + compaction, layer phases scaled to {w.n_layers} layers")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": v / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded)",
        "config": workload_config(w),
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "wall_s": wall}))


def workload_config(w, extra=None):
    c = {"workload": f"configs[{w.index - 1}] {w.name}: batch {w.batch}, {w.n_q_heads}q/{w.n_kv_heads}kv heads, "
                     f"head_dim {w.head_dim}, vocab {w.vocab}, prefix {w.prefix}, TT={w.tt} d={w.d} k={w.k}, "
                     f"{w.n_layers} layers of attention+compaction per step",
         "step": "tree_expand + n_layers x tree_attention + verify_accept + kv_compact(all layers)"}
    if extra:
        c.update(extra)
    return c


# ------------------------------------------------------------------------------ our arm
class DeviceWorkload:
    """All device state of one workload: a pool of distinct step inputs (each larger than
    L2 together with the per-layer KV caches) and the output buffers."""

    def __init__(self, w: synth.Workload, pool: int, seq_offset: int = 0):
        import torch
        from paper_2601_12212_b200 import binding
        self.torch, self.binding, self.w = torch, binding, w
        dev = "cuda"
        B, V, T, NL = w.batch, w.vocab, w.tt, w.n_layers
        self.B, self.T, self.pool = B, T, pool
        self.ctx = binding.Context(w.n_q_heads, w.n_kv_heads, w.head_dim, V, max_batch=B, max_tt=T,
                                   max_k=w.k, max_depth=w.d)
        i32 = dict(dtype=torch.int32, device=dev)
        self.L = [synth.initial_prefix(w, seq_offset + s) for s in range(B)]
        steps = np.array([[w.tt, w.d, w.k, self.L[s]] for s in range(B)], np.int32)
        self.h_steps = torch.from_numpy(steps).pin_memory()
        self.d_steps = self.h_steps.to(dev)
        self.d_steps_next = torch.zeros(B, 4, **i32)
        self.tokens = torch.zeros(B, T, **i32)
        self.parent = torch.zeros(B, T, **i32)
        self.depth = torch.zeros(B, T, **i32)
        self.pos = torch.zeros(B, T, **i32)
        self.mask = torch.zeros(B, T, 2, dtype=torch.int64, device=dev)
        self.retrieve = torch.zeros(B, T, w.d + 1, **i32)
        self.n_leaves = torch.zeros(B, **i32)
        self.n_nodes = torch.zeros(B, **i32)
        self.argmax = torch.zeros(B, T, **i32)
        self.path = torch.zeros(B, w.d + 1, **i32)
        self.alen = torch.zeros(B, **i32)
        self.out_tokens = torch.zeros(B, w.d + 1, **i32)
        self.result_host = torch.zeros(B, 2 * (w.d + 1) + 1, dtype=torch.int32).pin_memory()
        self.o = torch.zeros(B, T, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
        cap = w.kv_capacity
        self.cap = cap
        self.kv_strides = (w.n_kv_heads * cap * w.head_dim, cap * w.head_dim, w.head_dim)
        g = torch.Generator(device=dev)
        g.manual_seed(1234 + seq_offset)
        kv_shape = (B, w.n_kv_heads, cap, w.head_dim)
        # prefix and tree K/V: bf16 N(0,1).  (Timing only: values do not steer the data path of
        # attention; the parity tests use the host-seeded generators.)
        self.k = [torch.randn(kv_shape, generator=g, device=dev, dtype=torch.float32).bfloat16() for _ in range(NL)]
        self.v = [torch.randn(kv_shape, generator=g, device=dev, dtype=torch.float32).bfloat16() for _ in range(NL)]
        self.k_ptrs = binding.layer_pointer_table(self.k)
        self.v_ptrs = binding.layer_pointer_table(self.v)
        self.q = [torch.randn(B, T, w.n_q_heads, w.head_dim, generator=g, device=dev).bfloat16() for _ in range(NL)]
        # the pool of step inputs (host-seeded, pinned for the end-to-end leg)
        self.h_draft, self.h_target, self.h_root = [], [], []
        self.d_draft, self.d_target, self.d_root = [], [], []
        for i in range(pool):
            dl = np.stack([synth.draft_logits(w, i, seq_offset + s, w.d, w.k) for s in range(B)])
            roots = np.array([synth.root_token(w, i, seq_offset + s) for s in range(B)], np.int32)
            hd = torch.from_numpy(dl).pin_memory()
            hr = torch.from_numpy(roots).pin_memory()
            dd, dr = hd.to(dev), hr.to(dev)
            self.h_draft.append(hd), self.h_root.append(hr), self.d_draft.append(dd), self.d_root.append(dr)
            # the tree of this pool entry decides the target logits (the target "agrees" with a
            # child with probability p_agree); build it once with the library itself
            self.expand(i)
            torch.cuda.synchronize()
            tok, par, nn = self.tokens.cpu().numpy(), self.parent.cpu().numpy(), self.n_nodes.cpu().numpy()
            tl = np.zeros((B, T, V), np.float32)
            for s in range(B):
                tl[s, : nn[s]] = synth.target_logits(w, i, seq_offset + s, tok[s], par[s], int(nn[s]),
                                                     synth.agreement_prob(w, seq_offset + s))
            ht = torch.from_numpy(tl).pin_memory()
            self.h_target.append(ht), self.d_target.append(ht.to(dev))
        self.h_q = torch.stack([q.cpu() for q in self.q]).pin_memory()          # [NL][B][T][Hq][D]
        n0 = int(self.n_nodes[0])
        self.h_tree_kv = torch.randn(2, NL, B, w.n_kv_heads, T, w.head_dim).bfloat16().pin_memory()
        self.n0 = n0
        self.scale = 1.0 / float(np.sqrt(w.head_dim))

    # -- the four calls of a step ------------------------------------------------------
    def expand(self, i):
        w, V = self.w, self.w.vocab
        self.binding.resps_tree_expand(
            self.ctx, self.d_steps, self.B, self.d_draft[i], w.d * w.k * V, w.k * V, V, w.d, w.k,
            self.d_root[i], self.tokens, self.parent, self.depth, self.pos, self.mask, self.retrieve,
            self.n_leaves, self.n_nodes)

    def attention(self, l):
        self.binding.resps_tree_attention(
            self.ctx, self.d_steps, self.n_nodes, self.B, self.q[l], self.o, None, self.k[l], self.v[l],
            *self.kv_strides, self.cap, self.mask, self.scale)

    def verify(self, i):
        V = self.w.vocab
        self.binding.resps_verify_accept(
            self.ctx, self.d_steps, self.n_nodes, self.B, self.d_target[i], self.T * V, V, self.tokens,
            self.parent, self.argmax, self.path, self.alen, self.out_tokens, self.d_steps_next)

    def compact(self):
        self.binding.resps_kv_compact(self.ctx, self.d_steps, self.B, self.path, self.alen, self.k_ptrs,
                                      self.v_ptrs, self.w.n_layers, *self.kv_strides, self.cap)

    def step(self, i):
        self.expand(i)
        for l in range(self.w.n_layers):
            self.attention(l)
        self.verify(i)
        self.compact()

    LAUNCHES_PER_STEP = staticmethod(lambda w: 2 + 2 * w.n_layers + 2 + 1)  # scan, tree; attention + combine per layer; argmax, walk; compact

    # -- end to end: host buffers in, host result out ---------------------------------------
    def step_e2e(self, i):
        torch, w = self.torch, self.w
        L = self.L[0]
        self.d_steps.copy_(self.h_steps, non_blocking=True)
        self.d_root[i].copy_(self.h_root[i], non_blocking=True)
        self.d_draft[i].copy_(self.h_draft[i], non_blocking=True)
        self.d_target[i].copy_(self.h_target[i], non_blocking=True)
        for l in range(w.n_layers):
            self.q[l].copy_(self.h_q[l], non_blocking=True)
            for s in range(self.B):
                Ls = self.L[s]
                self.k[l][s, :, Ls:Ls + self.T].copy_(self.h_tree_kv[0, l, s], non_blocking=True)
                self.v[l][s, :, Ls:Ls + self.T].copy_(self.h_tree_kv[1, l, s], non_blocking=True)
        self.step(i)
        d1 = w.d + 1
        self.result_host[:, :d1].copy_(self.out_tokens, non_blocking=True)
        self.result_host[:, d1:2 * d1].copy_(self.path, non_blocking=True)
        self.result_host[:, 2 * d1].copy_(self.alen, non_blocking=True)

    def e2e_bytes(self):
        w = self.w
        h2d = (self.h_steps.numel() * 4 + self.h_root[0].numel() * 4 + self.h_draft[0].numel() * 4 +
               self.h_target[0].numel() * 4 + self.h_q.numel() * 2 + self.h_tree_kv.numel() * 2)
        d2h = self.result_host.numel() * 4
        return int(h2d), int(d2h)


def attention_algorithmic_bytes(w, L, n):
    """Per launch (one layer, one sequence): K and V of the L+n visible slots, Q in and O out."""
    return 2 * (L + n) * w.n_kv_heads * w.head_dim * 2 + 2 * n * w.n_q_heads * w.head_dim * 2


def max_over_ranks(values, world, device):
    """Device times of a multi-GPU run are reported as the maximum over the ranks (replicas run
    side by side, the job is as slow as its slowest rank); a single rank keeps its own."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_value(t_step_us, world):
    """us per speculative step of the whole job: `world` replicas finish one step each in t_step_us."""
    return t_step_us / world


def run_ours(args, w):
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    from paper_2601_12212_b200 import build
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()

    pool = 4
    dw = DeviceWorkload(w, pool, seq_offset=rank * w.batch)
    stream = torch.cuda.Stream()
    K, W = args.steps, max(3, args.warmup)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        # warm-up outside capture, then one captured graph per pool entry
        for i in range(pool):
            dw.step(i)
        torch.cuda.synchronize()
        graphs = []
        for i in range(pool):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                dw.step(i)
            graphs.append(g)
        attn_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(attn_graph, stream=stream):
            for l in range(w.n_layers):
                dw.attention(l)
        for i in range(W):
            graphs[i % pool].replay()
        barrier()

        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
        # ---- timed region 1: K whole steps, inputs resident in HBM -----------------------
        ev[0].record(stream)
        for i in range(K):
            graphs[i % pool].replay()
        ev[1].record(stream)
        barrier()
        # ---- timed region 2: the dominant kernel alone (all layers, back to back) ----------
        ev[2].record(stream)
        for i in range(K):
            attn_graph.replay()
        ev[3].record(stream)
        barrier()
        # ---- timed region 3: end to end from pinned host buffers ---------------------------
        for i in range(2):
            dw.step_e2e(i % pool)
        barrier()
        Ke = max(3, min(K, 20))
        ev[4].record(stream)
        for i in range(Ke):
            dw.step_e2e(i % pool)
        ev[5].record(stream)
        barrier()
        if rank == 0:
            # nvidia-smi delivers a sample every 100 ms and the timed regions are a few tens of ms: the
            # same step keeps running (untimed) until a handful of samples under this load are in
            t_stop = time.perf_counter() + 1.5
            i = 0
            while len(sampler.lines) < 6 and time.perf_counter() < t_stop:
                graphs[i % pool].replay()
                i += 1
                if i % 32 == 0:
                    torch.cuda.synchronize()
            torch.cuda.synchronize()
        clocks = sampler.stop() if rank == 0 else None

        t_step = ev[0].elapsed_time(ev[1]) * 1e3 / K            # us
        t_attn = ev[2].elapsed_time(ev[3]) * 1e3 / (K * w.n_layers)
        t_e2e = ev[4].elapsed_time(ev[5]) * 1e3 / Ke

        # per-phase breakdown (plain launches, not part of `value`)
        phases = {}
        for name, fn in (("expand", dw.expand), ("verify", dw.verify), ("compact", lambda r: dw.compact())):
            reps = 20
            fn(0)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for r in range(reps):
                fn(r % pool)
            b.record(stream)
            torch.cuda.synchronize()
            phases[name + "_us"] = a.elapsed_time(b) * 1e3 / reps

    t_step, t_attn, t_e2e = max_over_ranks([t_step, t_attn, t_e2e], world, "cuda")
    status = dw.ctx.status()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_src = measured_peaks()
    n = dw.n0
    L = dw.L[0]
    alg = attention_algorithmic_bytes(w, L, n) * w.batch
    achieved = alg / (t_attn * 1e-6) / 1e9
    V = w.vocab
    scan_bytes = (1 + (w.d - 1) * w.k) * V * 4 * w.batch
    argmax_bytes = n * V * 4 * w.batch
    h2d, d2h = dw.e2e_bytes()

    # CPU baseline: the oracle as it stands, one core, a bounded sample of the same workload
    cpu_layers = w.n_layers if w.index == 2 else 1
    t0 = time.perf_counter()
    parts = oracle_step_seconds(w, cpu_layers)
    cpu_wall = time.perf_counter() - t0
    cpu = {"value": oracle_us_per_step(w, parts), "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"one step: tree construction + verification in full, {cpu_layers} of {w.n_layers} "
                     f"layers of attention + compaction scaled to {w.n_layers} ({cpu_wall:.1f} s of CPU work)",
           "host_cores_available": os.cpu_count(),
           "phases_us": {"expand": parts["expand"] * 1e6, "attention_per_layer": parts["attn_per_layer"] * 1e6,
                         "verify": parts["verify"] * 1e6, "compact_per_layer": parts["compact_per_layer"] * 1e6}}

    line = {
        "metric": METRIC, "value": whole_job_value(t_step, world), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": t_step / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 attention (fp32 accumulate), fp32 logits", "data": "synthetic (seeded)",
        "config": workload_config(w, {
            "l2": f"inputs larger than L2: pool of {pool} distinct logit sets "
                  f"({(scan_bytes + argmax_bytes) * pool / 1e6:.0f} MB) and {w.n_layers} distinct KV-cache "
                  f"layers ({alg * w.n_layers / 1e6:.0f} MB read per step)",
            "launch": "CUDA graph of one whole step, replayed", "replicas": world,
            "n_nodes": n, "prefix_len": L}),
        "e2e": {"value": t_e2e / world, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": Ke},
        "gpu_launches": DeviceWorkload.LAUNCHES_PER_STEP(w) * K,
        "gpu_launches_per_step": DeviceWorkload.LAUNCHES_PER_STEP(w),
        "roofline": {"kernel": "tree_attention_kernel (+ attention_combine_kernel, one resps_tree_attention call)",
                     "bound": "hbm", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "traffic": ATTENTION_TRAFFIC_BYTES,
                     "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum of tree_attention_kernel, "
                                       "one launch of this workload (profiles/tree_attention_cfg2_ncu.md)",
                     "peak_source": peak_src, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                     "algorithmic_bytes_per_launch": alg, "us_per_launch": t_attn,
                     "launches_timed": K * w.n_layers},
        "phases": dict(phases, attention_per_layer_us=t_attn,
                       scan_gbs=scan_bytes / (phases["expand_us"] * 1e-6) / 1e9,
                       argmax_gbs=argmax_bytes / (phases["verify_us"] * 1e-6) / 1e9),
        "cpu_baseline": cpu, "clocks": clocks, "device_status": status,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=2, help="1-based index of the synthetic workload (synth.WORKLOADS)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    args = ap.parse_args()
    w = synth.WORKLOADS[args.config]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
