#!/usr/bin/env python
"""Benchmark of the speculative-step hot path (expand + attention over all layers + verify +
compaction) on seeded synthetic inputs shaped like the paper's target models.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference]

Prints ONE JSON line.  A step follows the chosen workload as stated: the per-step (TT, d, k) of its
schedule (each draw held for 4 steps where the workload says so), per-sequence prefixes, the model's
layer count, and the prefix growing by the accepted length ON THE DEVICE (the host writes no prefix
between steps).  `value` is microseconds per speculative step with all inputs resident in HBM,
measured with CUDA events around K replays of captured CUDA graphs of the step; `e2e` is the same
step driven from pinned HOST buffers (inputs copied in, results copied out inside the timed region);
`roofline` describes the dominant kernel (tree attention) from a live CUDA-event measurement,
`roofline_by_kernel` the three bandwidth-bound kernels; `cpu_baseline` is the CPU oracle timed on
this machine's host cores.  `--impl reference` times the CPU oracle alone.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
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
L2_BYTES = 126 * 1024 * 1024
# DRAM bytes per launch from profiler captures, kept beside their summaries: one record per
# (kernel, workload) with the bytes and the date of the capture; a record whose "kernel_rev" is not
# the current revision string of that kernel's source is stale and reported as null.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.json")


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return (float(j["hbm_gbs"]), float(j.get("bf16_tflops_sustained", 1400.0)),
                "measured (MEASURED_PEAKS.json hbm_gbs / bf16_tflops_sustained)")
    return 6650.0, 1400.0, "fallback (6.65 TB/s, 1.4 PFLOP/s sustained: earlier measurements on this pool)"


def kernel_rev(source: str) -> str:
    """Short content hash of a kernel source file: ties a stored profiler figure to the code it was taken from."""
    import hashlib
    path = os.path.join(ROOT, "paper_2601_12212_b200", "csrc", source)
    return hashlib.sha1(open(path, "rb").read()).hexdigest()[:12]


def recorded_traffic(kernel: str, workload_index: int, source: str):
    try:
        for rec in json.load(open(TRAFFIC_FILE))["records"]:
            if rec["kernel"] == kernel and rec["workload"] == workload_index:
                if rec.get("kernel_rev") == kernel_rev(source):
                    return rec["dram_bytes_per_launch"], rec.get("captured")
                return None, f"stale: taken from another revision of {source}"
    except (OSError, KeyError, ValueError):
        pass
    return None, "no capture on record"


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
def oracle_step_seconds(w: synth.Workload, attn_layers: int, step: int = 0, seqs=None):
    """One speculative step of the CPU oracle over the sequences `seqs` of the batch (all by default),
    with `attn_layers` of the workload's layers computed; returns per-phase seconds summed over those
    sequences.  Single-threaded C++ (see oracle/)."""
    import oracle
    seqs = range(w.batch) if seqs is None else seqs
    t_expand = t_attn = t_verify = t_compact = 0.0
    nodes = []
    for s in seqs:
        tt, d, k = synth.step_params(w, step, s)
        L = synth.initial_prefix(w, s)
        cap = L + tt + 8
        dl = synth.draft_logits(w, step, s, d, k)
        t0 = time.perf_counter()
        tree = oracle.tree_expand(synth.root_token(w, step, s), dl, tt, d, k, L)
        t_expand += time.perf_counter() - t0
        n = tree.n_nodes
        nodes.append(n)
        tl = synth.target_logits(w, step, s, tree.tokens, tree.parent, n, synth.agreement_prob(w, s))
        caches = []
        for l in range(attn_layers):
            kc = np.zeros((w.n_kv_heads, cap, w.head_dim), np.uint16)
            vc = np.zeros_like(kc)
            pk, pv = synth.prefix_kv(w, s, l, L)
            tk, tv = synth.tree_kv(w, step, s, l, n)
            kc[:, :L], vc[:, :L] = pk, pv
            kc[:, L:L + n], vc[:, L:L + n] = tk, tv
            q = synth.queries(w, step, s, l, n)
            t0 = time.perf_counter()
            oracle.tree_attention(q, kc, vc, L, tree.mask, 1.0 / np.sqrt(w.head_dim))
            t_attn += time.perf_counter() - t0
            caches.append((kc, vc))
        t0 = time.perf_counter()
        acc = oracle.verify_accept(tl, tree.tokens, tree.parent)
        t_verify += time.perf_counter() - t0
        t0 = time.perf_counter()
        for kc, vc in caches:
            oracle.kv_compact(kc, vc, L, acc.path)
        t_compact += time.perf_counter() - t0
    return {"expand": t_expand, "attn_per_layer": t_attn / max(1, attn_layers), "verify": t_verify,
            "compact_per_layer": t_compact / max(1, attn_layers), "n_nodes": nodes}


def oracle_us_per_step(w, parts, seq_scale=1.0):
    return 1e6 * seq_scale * (parts["expand"] + parts["verify"] +
                              w.n_layers * (parts["attn_per_layer"] + parts["compact_per_layer"]))


def oracle_sample_plan(w):
    """(layers, sequences) of one step the oracle is timed on: a bounded sample (about 10-30 s of CPU
    work), scaled to the workload's layer count and batch."""
    return {1: (1, None), 2: (w.n_layers, None), 3: (4, None), 4: (2, None), 5: (1, (0, 1, 2))}[w.index]


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    layers = 2 if w.index != 5 else 1
    seqs = None if w.index != 5 else (0,)
    seq_scale = 1.0 if seqs is None else w.batch / len(seqs)
    for i in range(args.warmup):
        oracle_step_seconds(w, 1, step=i, seqs=(0,))
    t0 = time.perf_counter()
    vals = [oracle_us_per_step(w, oracle_step_seconds(w, layers, step=i, seqs=seqs), seq_scale)
            for i in range(args.steps)]
    wall = time.perf_counter() - t0
    v = float(np.mean(vals))
    sample = (f"each of the {args.steps} timed steps computes tree construction + verification"
              f"{'' if seqs is None else f' of {len(seqs)} of the {w.batch} sequences'} in full and {layers} of the "
              f"{w.n_layers} layers' attention + compaction; the value scales the layer phases to {w.n_layers} layers"
              f"{'' if seqs is None else f' and everything to {w.batch} sequences'} "
              f"(measured on the sample: {wall / max(1, args.steps):.2f} s per step)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": v / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded)",
        "config": workload_config(w),
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "wall_s": wall, "measured_sample_s_per_step": wall / max(1, args.steps)}))


def workload_config(w):
    """The same for both arms: what is run, not how."""
    sched = (f"TT={w.tt} d={w.d} k={w.k}" if w.schedule == "fixed" else
             f"(TT,d,k) drawn per sequence from TT in {list(synth.GRID_TT)} x d in 3..8 x k in 4..12, held {w.hold} steps")
    return {"workload": f"configs[{w.index - 1}] {w.name}: batch {w.batch}, {w.n_q_heads}q/{w.n_kv_heads}kv heads, "
                        f"head_dim {w.head_dim}, vocab {w.vocab}, prefix {w.prefix} growing by the accepted length, "
                        f"{sched}, {w.n_layers} layers of attention+compaction per step",
            "step": "tree_expand + n_layers x tree_attention + verify_accept + kv_compact(all layers)"}


# ------------------------------------------------------------------------------ our arm
class DeviceWorkload:
    """All device state of one workload: a pool of step inputs (entry i = step i of the workload's
    schedule), the per-layer KV caches and the output buffers.  The step parameters live in device
    memory; the prefix length advances there (resps_verify_accept writes it back in place)."""

    def __init__(self, w: synth.Workload, pool: int, seq_offset: int = 0):
        import torch
        from paper_2601_12212_b200 import binding
        self.torch, self.binding, self.w = torch, binding, w
        dev = "cuda"
        grid = w.schedule == "grid"
        self.T = T = max(synth.GRID_TT) if grid else w.tt
        self.max_k = max(synth.GRID_K) if grid else w.k
        self.max_d = max(synth.GRID_D) if grid else w.d
        B, V, NL = w.batch, w.vocab, w.n_layers
        self.B, self.pool, self.seq_offset = B, pool, seq_offset
        self.ctx = binding.Context(w.n_q_heads, w.n_kv_heads, w.head_dim, V, max_batch=B, max_tt=T,
                                   max_k=self.max_k, max_depth=self.max_d)
        i32 = dict(dtype=torch.int32, device=dev)
        self.L0 = [synth.initial_prefix(w, seq_offset + s) for s in range(B)]
        self.params = [[synth.step_params(w, i, seq_offset + s) for s in range(B)] for i in range(pool)]
        steps0 = np.array([[*self.params[0][s], self.L0[s]] for s in range(B)], np.int32)
        self.h_steps0 = torch.from_numpy(steps0).pin_memory()
        self.d_steps = self.h_steps0.to(dev)
        self.h_params = [torch.from_numpy(np.array(p, np.int32)).pin_memory() for p in self.params]
        self.d_params = [h.to(dev) for h in self.h_params]
        self.tokens = torch.zeros(B, T, **i32)
        self.parent = torch.zeros(B, T, **i32)
        self.depth = torch.zeros(B, T, **i32)
        self.pos = torch.zeros(B, T, **i32)
        self.mask = torch.zeros(B, T, 2, dtype=torch.int64, device=dev)
        self.retrieve = torch.zeros(B, T, self.max_d + 1, **i32)
        self.n_leaves = torch.zeros(B, **i32)
        self.n_nodes = torch.zeros(B, **i32)
        self.argmax = torch.zeros(B, T, **i32)
        self.path = torch.zeros(B, self.max_d + 1, **i32)
        self.alen = torch.zeros(B, **i32)
        self.out_tokens = torch.zeros(B, self.max_d + 1, **i32)
        self.result_host = torch.zeros(B, 2 * (self.max_d + 1) + 1, dtype=torch.int32).pin_memory()
        self.o = torch.zeros(B, T, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
        cap = w.kv_capacity
        self.cap = cap
        self.kv_strides = (w.n_kv_heads * cap * w.head_dim, cap * w.head_dim, w.head_dim)
        g = torch.Generator(device=dev)
        g.manual_seed(1234 + seq_offset)
        kv_shape = (B, w.n_kv_heads, cap, w.head_dim)
        # prefix and tree K/V: bf16 N(0,1) in every slot, so that whatever the prefix has grown to the
        # tree tokens' K/V "are already there".  (Timing only: values do not steer the data path of
        # attention; the parity tests use the host-seeded generators.)
        self.k = [torch.randn(kv_shape, generator=g, device=dev, dtype=torch.bfloat16) for _ in range(NL)]
        self.v = [torch.randn(kv_shape, generator=g, device=dev, dtype=torch.bfloat16) for _ in range(NL)]
        self.k_ptrs = binding.layer_pointer_table(self.k)
        self.v_ptrs = binding.layer_pointer_table(self.v)
        self.q = [torch.randn(B, T, w.n_q_heads, w.head_dim, generator=g, device=dev, dtype=torch.bfloat16)
                  for _ in range(NL)]
        # the pool of step inputs (host-seeded, pinned for the end-to-end leg)
        self.h_draft, self.h_target, self.h_root = [], [], []
        self.d_draft, self.d_target, self.d_root = [], [], []
        self.nodes = []
        for i in range(pool):
            dl = np.zeros((B, self.max_d, self.max_k, V), np.float32)
            for s in range(B):
                tt, d, k = self.params[i][s]
                dl[s, :d, :k] = synth.draft_logits(w, i, seq_offset + s, d, k)
            roots = np.array([synth.root_token(w, i, seq_offset + s) for s in range(B)], np.int32)
            hd = torch.from_numpy(dl).pin_memory()
            hr = torch.from_numpy(roots).pin_memory()
            self.h_draft.append(hd), self.h_root.append(hr)
            self.d_draft.append(hd.to(dev)), self.d_root.append(hr.to(dev))
            # the tree of this pool entry decides the target logits (the target "agrees" with a
            # child with probability p_agree); build it once with the library itself
            self.set_params(i)
            self.expand(i)
            torch.cuda.synchronize()
            tok, par, nn = self.tokens.cpu().numpy(), self.parent.cpu().numpy(), self.n_nodes.cpu().numpy()
            tl = np.zeros((B, T, V), np.float32)
            for s in range(B):
                tl[s, : nn[s]] = synth.target_logits(w, i, seq_offset + s, tok[s], par[s], int(nn[s]),
                                                     synth.agreement_prob(w, seq_offset + s))
            ht = torch.from_numpy(tl).pin_memory()
            self.h_target.append(ht), self.d_target.append(ht.to(dev))
            self.nodes.append([int(x) for x in nn])
        self.h_q = torch.stack([q.cpu() for q in self.q]).pin_memory()          # [NL][B][T][Hq][D]
        self.h_tree_kv = torch.randn(2, NL, B, w.n_kv_heads, T, w.head_dim).bfloat16().pin_memory()
        self.scale = 1.0 / float(np.sqrt(w.head_dim))
        # uniforms for the acceptance under sampling (timed as a phase of its own, not part of the step)
        self.u_accept = torch.rand(B, self.max_d + 1, self.max_k, generator=g, device=dev, dtype=torch.float64)
        self.u_sample = torch.rand(B, self.max_d + 1, generator=g, device=dev, dtype=torch.float64)
        self.reset_prefix()

    def reset_prefix(self):
        """Back to step 0's parameters and the initial prefix lengths (outside any timed region)."""
        self.d_steps.copy_(self.h_steps0)
        self.host_L = list(self.L0)

    def steps_until_overflow(self):
        grow = self.max_d + 1
        return min((self.cap - L - self.T) // grow for L in self.L0)

    # -- the calls of a step ------------------------------------------------------------
    def set_params(self, i):
        """(TT, d, k) of pool entry i into the device-resident step array; the prefix column stays."""
        self.d_steps[:, :3].copy_(self.d_params[i])

    def expand(self, i):
        V = self.w.vocab
        self.binding.resps_tree_expand(
            self.ctx, self.d_steps, self.B, self.d_draft[i], self.max_d * self.max_k * V, self.max_k * V, V,
            self.max_d, self.max_k, self.d_root[i], self.tokens, self.parent, self.depth, self.pos, self.mask,
            self.retrieve, self.n_leaves, self.n_nodes)

    def attention(self, l):
        self.binding.resps_tree_attention(
            self.ctx, self.d_steps, self.n_nodes, self.B, self.q[l], self.o, None, self.k[l], self.v[l],
            *self.kv_strides, self.cap, self.mask, self.scale)

    def verify(self, i, advance=True):
        V = self.w.vocab
        self.binding.resps_verify_accept(
            self.ctx, self.d_steps, self.n_nodes, self.B, self.d_target[i], self.T * V, V, self.tokens,
            self.parent, self.argmax, self.path, self.alen, self.out_tokens,
            self.d_steps if advance else None)

    def verify_sampled(self, i, temperature=1.0):
        V = self.w.vocab
        self.binding.resps_verify_accept_sampled(
            self.ctx, self.d_steps, self.n_nodes, self.B, self.d_target[i], self.T * V, V, self.d_draft[i],
            self.max_d * self.max_k * V, self.max_k * V, V, temperature, self.tokens, self.parent, self.u_accept,
            self.u_sample, self.path, self.alen, self.out_tokens, None)

    def compact(self, advanced=True):
        self.binding.resps_kv_compact(self.ctx, self.d_steps, self.B, self.path, self.alen, self.k_ptrs,
                                      self.v_ptrs, self.w.n_layers, *self.kv_strides, self.cap,
                                      steps_advanced=advanced)

    def prime(self, i):
        """The step array as the step before pool entry i leaves it (entries follow one another cyclically)."""
        self.set_params((i - 1) % self.pool)

    def step(self, i):
        # (TT, d, k) are rewritten only when the schedule changes them, as a controller would
        if self.params[i] != self.params[(i - 1) % self.pool]:
            self.set_params(i)
        self.expand(i)
        for l in range(self.w.n_layers):
            self.attention(l)
        self.verify(i)          # prefix_len += accepted + 1, in place on the device
        self.compact()

    def launches_per_step(self):
        # scan, tree build; the attention work list once; attention + combine per layer; arg-max with the walk
        # in its tail; compaction (the launch list under profiles/ shows the same 69 per step at 32 layers)
        return 2 + 1 + 2 * self.w.n_layers + 1 + 1

    # -- end to end: host buffers in, host result out ---------------------------------------
    def step_e2e(self, i):
        """One host-driven step: this step's inputs go up from pinned memory, the kernels run, the
        accepted tokens and path come back and the host waits for them (it needs them to prepare the
        next step, here: to know where the next tree's K/V go)."""
        torch, w = self.torch, self.w
        self.d_steps[:, :3].copy_(self.h_params[i], non_blocking=True)
        self.d_root[i].copy_(self.h_root[i], non_blocking=True)
        self.d_draft[i].copy_(self.h_draft[i], non_blocking=True)
        self.d_target[i].copy_(self.h_target[i], non_blocking=True)
        for l in range(w.n_layers):
            self.q[l].copy_(self.h_q[l], non_blocking=True)
            for s in range(self.B):
                Ls = self.host_L[s]
                self.k[l][s, :, Ls:Ls + self.T].copy_(self.h_tree_kv[0, l, s], non_blocking=True)
                self.v[l][s, :, Ls:Ls + self.T].copy_(self.h_tree_kv[1, l, s], non_blocking=True)
        self.expand(i)
        for l in range(w.n_layers):
            self.attention(l)
        self.verify(i)
        self.compact()
        d1 = self.max_d + 1
        self.result_host[:, :d1].copy_(self.out_tokens, non_blocking=True)
        self.result_host[:, d1:2 * d1].copy_(self.path, non_blocking=True)
        self.result_host[:, 2 * d1].copy_(self.alen, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        for s in range(self.B):
            self.host_L[s] += int(self.result_host[s, 2 * d1]) + 1

    def e2e_bytes(self):
        h2d = (self.h_params[0].numel() * 4 + self.h_root[0].numel() * 4 + self.h_draft[0].numel() * 4 +
               self.h_target[0].numel() * 4 + self.h_q.numel() * 2 + self.h_tree_kv.numel() * 2)
        d2h = self.result_host.numel() * 4
        return int(h2d), int(d2h)


def measure_widened_rows(dw, w, stream, flush):
    """Device time of the calls beyond the four of a step (not part of `value`): the level form of the tree
    expansion, the vocabulary split over two ranks (one rank's calls; the two small all-gathers are the caller's
    and are not timed) and the controller step.  Each figure is the mean of three cold calls after an L2 flush."""
    import torch
    binding = dw.binding
    B, V, T, MK, MD = dw.B, w.vocab, dw.T, dw.max_k, dw.max_d
    i32 = dict(dtype=torch.int32, device="cuda")
    out = {}

    def timed(fn, reps=3):
        fn()
        torch.cuda.synchronize()
        total = 0.0
        for rep in range(reps):
            flush.fill_(rep)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            torch.cuda.synchronize()
            total += a.elapsed_time(b) * 1e3
        return total / reps

    dw.reset_prefix()
    dw.set_params(0)
    d_max = max(d for (_, d, _) in dw.params[0])
    tree_out = (dw.tokens, dw.parent, dw.depth, dw.pos, dw.mask, dw.retrieve, dw.n_leaves, dw.n_nodes)
    # ---- level form: begin, one call per level (the draft model would run in between), finish ----------
    f_tok, f_par, f_pos, f_idx = (torch.zeros(B, MK, **i32) for _ in range(4))
    f_mask = torch.zeros(B, MK, 2, dtype=torch.int64, device="cuda")
    dflat, tflat = dw.d_draft[0].view(-1), dw.d_target[0].view(-1)

    def level_form():
        binding.resps_tree_expand_begin(dw.ctx, dw.d_steps, B, MK)
        for j in range(d_max):
            binding.resps_tree_expand_level(dw.ctx, dw.d_steps, B, j, dflat[j * MK * V:], MD * MK * V, V,
                                            f_tok, f_par, f_pos, f_idx, f_mask, None)
        binding.resps_tree_expand_finish(dw.ctx, dw.d_steps, B, dw.d_root[0], *tree_out)
    out["expand_level_form_us"] = timed(level_form)
    out["expand_level_form_calls"] = d_max + 2
    # ---- vocabulary split over two ranks: what rank 0 runs ------------------------------------------------
    P = 2
    cols = binding.shard_columns(V, P)
    ctxs = [binding.Context(w.n_q_heads, w.n_kv_heads, w.head_dim, wd, max_batch=B, max_tt=T, max_k=MK, max_depth=MD)
            for _, wd in cols]
    rows = int(binding.load().resps_scan_rows(ctxs[0].handle))
    d_off = torch.tensor([off for off, _ in cols], **i32)
    parts = [(torch.zeros(B, rows, MK, device="cuda"), torch.zeros(B, rows, MK, **i32),
              torch.zeros(B, rows, dtype=torch.float64, device="cuda")) for _ in range(P)]
    keys = [torch.zeros(B, T, dtype=torch.int64, device="cuda") for _ in range(P)]
    for p_, (off, wd) in enumerate(cols):          # the other rank's share, outside the timing
        binding.resps_row_scan_shard(ctxs[p_], dw.d_steps, B, dflat[off:], MD * MK * V, MK * V, V, MD, MK, *parts[p_])
    all_parts = [torch.stack([parts[p_][i] for p_ in range(P)]) for i in range(3)]

    def sharded_expand():
        binding.resps_row_scan_shard(ctxs[0], dw.d_steps, B, dflat, MD * MK * V, MK * V, V, MD, MK, *parts[0])
        binding.resps_tree_expand_merge(ctxs[0], dw.d_steps, B, MD, MK, P, *all_parts, d_off, dw.d_root[0], *tree_out)
    out["expand_vocab_2way_rank_us"] = timed(sharded_expand)
    for p_, (off, wd) in enumerate(cols):
        binding.resps_target_argmax_shard(ctxs[p_], dw.n_nodes, B, tflat[off:], T * V, V, keys[p_])
    all_keys = torch.stack(keys)

    def sharded_verify():
        binding.resps_target_argmax_shard(ctxs[0], dw.n_nodes, B, tflat, T * V, V, keys[0])
        binding.resps_verify_accept_merge(ctxs[0], dw.d_steps, dw.n_nodes, B, P, all_keys, d_off, dw.tokens, dw.parent,
                                          dw.argmax, dw.path, dw.alen, dw.out_tokens, None)
    out["verify_vocab_2way_rank_us"] = timed(sharded_verify)
    for c in ctxs:
        c.close()
    # ---- controller step: the [128,128] policy on three hidden layers of the model's width, asked every call ------
    hidden = w.n_q_heads * w.head_dim
    actions = torch.tensor(synth.action_space(filtered=True), **i32)
    A, H, F = actions.shape[0], 128, 3 * hidden
    g = torch.Generator(device="cuda").manual_seed(1)
    rnd = lambda *shape: torch.randn(*shape, device="cuda", generator=g)
    pol = binding.make_policy(rnd(H, F) / F ** 0.5, rnd(H) * 0.1, rnd(H, H) / H ** 0.5, rnd(H) * 0.1, rnd(A, H) * 0.5,
                              rnd(A) * 0.1, actions)
    hid = [rnd(B, hidden).bfloat16() for _ in range(3)]
    c_state = torch.zeros(B, 4, **i32)
    c_steps = dw.d_steps.clone()
    c_reward = torch.zeros(B, device="cuda")
    c_u = torch.full((B,), 0.5, dtype=torch.float64, device="cuda")
    c_ctx = binding.Context(w.n_q_heads, w.n_kv_heads, w.head_dim, 1024, max_batch=B, max_tt=128, max_k=32, max_depth=8)

    def controller():
        binding.resps_controller_step(c_ctx, pol, *hid, hidden, B, 1, 0.0, c_u, None, None, c_state, c_steps, c_reward)
    out["controller_step_us"] = timed(controller)
    out["controller_step_bytes"] = H * F * 4 + 3 * B * hidden * 2
    c_ctx.close()
    dw.reset_prefix()
    return out


def attention_algorithmic(w, Ls, ns):
    """Per launch (one layer, the whole batch): K and V of the L+n visible slots, Q in and O out (bytes);
    4 n Hq (L+n) D flop."""
    by = sum(2 * (L + n) * w.n_kv_heads * w.head_dim * 2 + 2 * n * w.n_q_heads * w.head_dim * 2 for L, n in zip(Ls, ns))
    fl = sum(4 * n * w.n_q_heads * (L + n) * w.head_dim for L, n in zip(Ls, ns))
    return by, fl


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


def pool_size(w):
    """Distinct step inputs kept on the device: at least 4, and enough logits between two uses of
    the same entry to exceed L2 several times where memory allows."""
    grid = w.schedule == "grid"
    max_d, max_k, T = (max(synth.GRID_D), max(synth.GRID_K), max(synth.GRID_TT)) if grid else (w.d, w.k, w.tt)
    per_entry = w.batch * (max_d * max_k + T) * w.vocab * 4
    return int(min(16, max(4, -(-3 * L2_BYTES // per_entry))))


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

    pool = pool_size(w)
    dw = DeviceWorkload(w, pool, seq_offset=rank * w.batch)
    stream = torch.cuda.Stream()
    W = max(3, args.warmup)
    K = max(1, min(args.steps, dw.steps_until_overflow() - W - 2))
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")

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
        # `pool` consecutive steps as one graph, in the order the timed region takes them: the gap between
        # two graph launches (20-25 us of idle GPU on this pool) is then paid once per `pool` steps
        multi = torch.cuda.CUDAGraph()
        with torch.cuda.graph(multi, stream=stream):
            for j in range(pool):
                dw.step((W + j) % pool)
        # the dominant kernel alone: all layers of one step, back to back, on the tree of pool entry 0
        dw.reset_prefix()
        dw.set_params(0)
        dw.expand(0)
        torch.cuda.synchronize()
        attn_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(attn_graph, stream=stream):
            for l in range(w.n_layers):
                dw.attention(l)
        attn_graph.replay()
        dw.reset_prefix()
        dw.prime(W % pool)
        multi.replay()  # first launch of the multi-step graph (uploads it); the prefix is reset again below
        torch.cuda.synchronize()
        dw.reset_prefix()
        for i in range(W):
            graphs[i % pool].replay()
        barrier()

        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
        # ---- timed region 1: K whole steps, inputs resident in HBM; the prefix advances on the device ----
        ev[0].record(stream)
        for _ in range(K // pool):
            multi.replay()
        for i in range(K - K % pool, K):
            graphs[(W + i) % pool].replay()
        ev[1].record(stream)
        barrier()
        prefix_after = [int(x) for x in dw.d_steps[:, 3].cpu()]
        # ---- timed region 2: the dominant kernel alone (all layers, back to back) ----------
        dw.reset_prefix()
        dw.set_params(0)
        dw.expand(0)
        torch.cuda.synchronize()
        Ka = max(1, min(K, 2000 // w.n_layers))
        ev[2].record(stream)
        for i in range(Ka):
            attn_graph.replay()
        ev[3].record(stream)
        barrier()
        attn_L = [int(x) for x in dw.d_steps[:, 3].cpu()]
        attn_n = [int(x) for x in dw.n_nodes.cpu()]
        # ---- timed region 3: end to end from pinned host buffers ---------------------------
        dw.reset_prefix()
        for i in range(2):
            dw.step_e2e(i % pool)
        barrier()
        Ke = max(3, min(K, 20))
        ev[4].record(stream)
        for i in range(Ke):
            dw.step_e2e((2 + i) % pool)
        ev[5].record(stream)
        barrier()
        if rank == 0:
            # nvidia-smi delivers a sample every 100 ms and the timed regions are a few tens of ms: the
            # same step keeps running (untimed) until a handful of samples under this load are in
            t_stop = time.perf_counter() + 1.5
            i = 0
            dw.reset_prefix()
            while len(sampler.lines) < 6 and time.perf_counter() < t_stop:
                graphs[i % pool].replay()
                i += 1
                if i % 32 == 0:
                    torch.cuda.synchronize()
                    dw.reset_prefix()
            torch.cuda.synchronize()
        clocks = sampler.stop() if rank == 0 else None

        t_step = ev[0].elapsed_time(ev[1]) * 1e3 / K            # us
        t_attn = ev[2].elapsed_time(ev[3]) * 1e3 / (Ka * w.n_layers)
        t_e2e = ev[4].elapsed_time(ev[5]) * 1e3 / Ke

        # per-phase figures (not part of `value`): each call alone between two events, L2 flushed before
        # it (a 252 MB fill), summed over the pool entries
        dw.reset_prefix()
        phases, phase_bytes = {}, {}
        for name, fn in (("expand", dw.expand), ("verify", lambda i: dw.verify(i, advance=False)),
                         ("verify_sampled_t1", dw.verify_sampled), ("compact", lambda i: dw.compact(advanced=False))):
            fn(0)
            torch.cuda.synchronize()
            total, reps = 0.0, 0
            for rep in range(3):
                for i in range(pool):
                    if name != "compact":
                        dw.set_params(i)
                        if name != "expand":
                            dw.expand(i)
                    flush.fill_(rep)
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(stream)
                    fn(i)
                    b.record(stream)
                    torch.cuda.synchronize()
                    total += a.elapsed_time(b) * 1e3
                    reps += 1
            phases[name + "_us"] = total / reps
        # the same calls as they run inside a step: a replayed graph of one call per pool entry, back to
        # back (distinct logits every call, more than L2 in total; no flush, no host launch in between)
        in_sequence = {}
        same_params = all(dw.params[i] == dw.params[0] for i in range(pool))
        for name in ("expand", "verify"):
            dw.reset_prefix()
            dw.set_params(0)
            dw.expand(0)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for i in range(pool):
                    if name == "expand":
                        if not same_params:
                            dw.set_params(i)
                        dw.expand(i)
                    else:
                        dw.verify(i, advance=False)  # the tree of entry 0 against the target rows of entry i
            for _ in range(2):
                g.replay()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(3):
                g.replay()
            b.record(stream)
            torch.cuda.synchronize()
            in_sequence[name + "_us"] = a.elapsed_time(b) * 1e3 / (3 * pool)
        widened = None
        if rank == 0:
            try:
                widened = measure_widened_rows(dw, w, stream, flush)
            except Exception as e:  # these figures are extras: the line is printed without them
                widened = {"error": f"{type(e).__name__}: {e}"}
        V = w.vocab
        phase_bytes["scan"] = float(np.mean([sum((1 + (d - 1) * k) * V * 4 for (_, d, k) in dw.params[i])
                                             for i in range(pool)]))
        phase_bytes["argmax"] = float(np.mean([sum(dw.nodes[i]) * V * 4 for i in range(pool)]))

        if args.step_log and rank == 0:
            # untimed extra pass: every step between its own pair of events, one JSON line per step
            dw.reset_prefix()
            dw.prime(W % pool)
            torch.cuda.synchronize()
            pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
            for i, (a, b) in enumerate(pairs):
                a.record(stream)
                graphs[(W + i) % pool].replay()
                b.record(stream)
            torch.cuda.synchronize()
            with open(args.step_log, "w") as f:
                for i, (a, b) in enumerate(pairs):
                    e = (W + i) % pool
                    f.write(json.dumps({"step": i, "us": a.elapsed_time(b) * 1e3, "pool_entry": e,
                                        "tt_d_k": [list(p) for p in dw.params[e]], "n_nodes": list(dw.nodes[e])}) + "\n")

    t_step, t_attn, t_e2e = max_over_ranks([t_step, t_attn, t_e2e], world, "cuda")
    status = dw.ctx.status()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    hbm_peak, tensor_peak, peak_src = measured_peaks()
    alg_bytes, alg_flop = attention_algorithmic(w, attn_L, attn_n)
    achieved = alg_bytes / (t_attn * 1e-6) / 1e9
    tflops = alg_flop / (t_attn * 1e-6) / 1e12
    # the roof that binds the attention launch: the slower of its HBM time and its tensor-pipe time
    t_hbm, t_tensor = alg_bytes / (hbm_peak * 1e9), alg_flop / (tensor_peak * 1e12)
    bound = "hbm" if t_hbm >= t_tensor else "tensor"
    h2d, d2h = dw.e2e_bytes()
    traffic, traffic_note = recorded_traffic("tree_attention_kernel", w.index, "attention.cu")

    def hbm_entry(kernel, by, us, note):
        gbs = by / (us * 1e-6) / 1e9
        return {"kernel": kernel, "bound": "hbm", "algorithmic_bytes": by, "us": us, "achieved": gbs, "unit": "GB/s",
                "peak": hbm_peak, "frac": gbs / hbm_peak, "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS, "timing": note}

    by_kernel = [
        dict(hbm_entry("tree_attention_kernel (one resps_tree_attention call, whole batch)", alg_bytes, t_attn,
                       "CUDA events around a replayed graph of all layers, back to back"),
             flop=alg_flop, tflops=tflops,
             binding_roof=bound,
             frac_of_binding_roof=(achieved / hbm_peak if bound == "hbm" else tflops / tensor_peak),
             tensor_peak_tflops=tensor_peak),
        hbm_entry("row_scan_stream_kernel + tree_build_kernel (one resps_tree_expand call)", phase_bytes["scan"],
                  phases["expand_us"], "one call between two events after an L2 flush, mean over the pool"),
        hbm_entry("row_argmax_stream_kernel with the acceptance walk in its tail (one resps_verify_accept call)", phase_bytes["argmax"],
                  phases["verify_us"], "one call between two events after an L2 flush, mean over the pool"),
        hbm_entry("row_scan_stream_kernel + tree_build_kernel (one resps_tree_expand call)", phase_bytes["scan"],
                  in_sequence["expand_us"], "replayed graph of one call per pool entry, back to back"),
        hbm_entry("row_argmax_stream_kernel with the acceptance walk in its tail (one resps_verify_accept call)", phase_bytes["argmax"],
                  in_sequence["verify_us"], "replayed graph of one call per pool entry, back to back"),
    ]

    # CPU baseline: the oracle as it stands, one core, a bounded sample of the same workload
    cpu_layers, cpu_seqs = oracle_sample_plan(w)
    seq_scale = 1.0 if cpu_seqs is None else w.batch / len(cpu_seqs)
    t0 = time.perf_counter()
    parts = oracle_step_seconds(w, cpu_layers, seqs=cpu_seqs)
    cpu_wall = time.perf_counter() - t0
    cpu = {"value": oracle_us_per_step(w, parts, seq_scale), "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"step 0: tree construction + verification in full"
                     f"{'' if cpu_seqs is None else f' for {len(cpu_seqs)} of {w.batch} sequences'}, {cpu_layers} of "
                     f"{w.n_layers} layers of attention + compaction; scaled to {w.n_layers} layers"
                     f"{'' if cpu_seqs is None else f' and {w.batch} sequences'} ({cpu_wall:.1f} s of CPU work)",
           "host_cores_available": os.cpu_count(),
           "phases_us": {"expand": parts["expand"] * 1e6 * seq_scale,
                         "attention_per_layer": parts["attn_per_layer"] * 1e6 * seq_scale,
                         "verify": parts["verify"] * 1e6 * seq_scale,
                         "compact_per_layer": parts["compact_per_layer"] * 1e6 * seq_scale}}

    line = {
        "metric": METRIC, "value": whole_job_value(t_step, world), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": t_step / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 attention (fp32 accumulate), fp32 logits", "data": "synthetic (seeded)",
        "config": workload_config(w),
        "run": {"l2": f"inputs larger than L2: pool of {pool} distinct step inputs "
                      f"({(phase_bytes['scan'] + phase_bytes['argmax']) * pool / 1e6:.0f} MB of logits) and {w.n_layers} "
                      f"distinct KV-cache layers ({alg_bytes * w.n_layers / 1e6:.0f} MB read per step)",
                "launch": f"CUDA graphs, replayed: one of {pool} consecutive whole steps ({K // pool} replays) and "
                          f"single-step graphs for the remaining {K % pool} steps; step parameters and prefix "
                          "lengths live in device memory and the prefix advances there",
                "replicas": world, "pool": pool, "prefix_start": dw.L0, "prefix_after_timed_steps": prefix_after,
                "n_nodes_per_pool_entry": dw.nodes[:4]},
        "e2e": {"value": t_e2e / world, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": Ke},
        "gpu_launches": dw.launches_per_step() * K,
        "gpu_launches_per_step": dw.launches_per_step(),
        "roofline": {"kernel": "tree_attention_kernel (one resps_tree_attention call)",
                     "bound": bound, "achieved": achieved if bound == "hbm" else tflops,
                     "peak": hbm_peak if bound == "hbm" else tensor_peak,
                     "unit": "GB/s" if bound == "hbm" else "TFLOP/s",
                     "frac": achieved / hbm_peak if bound == "hbm" else tflops / tensor_peak,
                     "traffic": traffic, "traffic_source": traffic_note,
                     "peak_source": peak_src, "hbm_gbs": achieved, "hbm_frac_of_measured": achieved / hbm_peak,
                     "hbm_frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS, "tflops": tflops,
                     "algorithmic_bytes_per_launch": alg_bytes, "algorithmic_flop_per_launch": alg_flop,
                     "us_per_launch": t_attn, "launches_timed": Ka * w.n_layers,
                     "prefix_len": attn_L, "n_nodes": attn_n},
        "roofline_by_kernel": by_kernel,
        "phases": dict(phases, attention_per_layer_us=t_attn),
        "phases_in_sequence": dict(in_sequence, note="one call per pool entry in a replayed graph, back to back: "
                                   "the cost of the call inside a step; `phases` times single cold calls"),
        "widened_rows": widened,
        "cpu_baseline": cpu, "clocks": clocks, "device_status": status,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=2, help="1-based index of the synthetic workload (synth.WORKLOADS)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--step-log", default=None, metavar="FILE",
                    help="also write one JSON line per step (device time, step parameters, tree sizes) from an "
                         "untimed extra pass")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.config]
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under a launcher: start one replica per GPU ourselves
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    if world != args.gpus:
        sys.exit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}: start it with one rank per GPU "
                 f"(or without a launcher, then it starts the ranks itself)")
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
