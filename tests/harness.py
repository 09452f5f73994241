"""Test harness: drives the CUDA library through the C-ABI binding step by step on a seeded
synthetic workload and compares every output with the CPU oracle on the same inputs.
Test infrastructure only (it imports the oracle)."""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

import oracle
from paper_2601_12212_b200 import binding, synth

TAU = 1e-4          # fp64 score gap below which a selection boundary counts as a near tie
ATTN_ABS = 2e-2     # max abs error of attention outputs (bf16 in, fp32 accumulate)
ATTN_REL = 1e-2     # max error relative to max(|o|, rms of the output row)
# log-sum-exp of the scaled scores, fp32 on the GPU: the scores are exact bf16 products summed in
# fp32 (relative 2^-24 per add over D terms), ex2.approx is 2 ulp and the running sum is fp32, so the
# sum of up to 2^14 terms is within ~2^-24 * 2^7 (random-walk) .. 2^-24 * 2^14 (worst case) = 1e-3
# relative, i.e. 1e-3 absolute on its logarithm; partial combines add a handful of fp32 roundings.
LSE_ABS = 2e-3


def u16_to_bf16_cuda(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy().astype(np.float64)


def check_attention(gpu: np.ndarray, ref: np.ndarray):
    """gpu, ref: fp64 [n][Hq][D]. Returns (max abs err, max rel err) and asserts both gates."""
    err = np.abs(gpu - ref)
    rms = np.sqrt((ref * ref).mean(axis=-1, keepdims=True))
    rel = err / np.maximum(np.abs(ref), rms)
    a, r = float(err.max()), float(rel.max())
    assert a <= ATTN_ABS, f"attention max abs err {a}"
    assert r <= ATTN_REL, f"attention max rel err {r}"
    return a, r


@dataclass
class Stats:
    steps: int = 0
    near_tie_steps: int = 0      # (step, sequence) pairs with a selection-boundary gap below TAU
    near_tie_swaps: list = field(default_factory=list)  # (step, seq, flipped pairs) accepted as a swap within TAU
    attn_checks: int = 0
    attn_max_abs: float = 0.0
    attn_max_rel: float = 0.0
    accept_lens: list = field(default_factory=list)
    n_nodes: list = field(default_factory=list)


class Runner:
    """Holds device + host state of one workload and runs whole steps with parity checks."""

    def __init__(self, w: synth.Workload, n_layers: int = 1, kv_capacity: int | None = None,
                 max_tt: int | None = None):
        self.w = w
        self.B = w.batch
        self.nl = n_layers
        self.cap = kv_capacity or w.kv_capacity
        grid = w.schedule == "grid"
        self.max_k = max(synth.GRID_K) if grid else w.k
        self.max_d = max(synth.GRID_D) if grid else w.d
        self.max_tt = max_tt or (max(synth.GRID_TT) if grid else w.tt)
        self.ctx = binding.Context(w.n_q_heads, w.n_kv_heads, w.head_dim, w.vocab, max_batch=self.B,
                                   max_tt=self.max_tt, max_k=self.max_k, max_depth=self.max_d)
        dev = "cuda"
        B, T, V = self.B, self.max_tt, w.vocab
        i32 = dict(dtype=torch.int32, device=dev)
        self.d_steps = torch.zeros(B, 4, **i32)
        self.d_steps_next = torch.zeros(B, 4, **i32)
        self.d_root = torch.zeros(B, **i32)
        self.d_draft = torch.zeros(B, self.max_d, self.max_k, V, dtype=torch.float32, device=dev)
        self.d_tokens = torch.full((B, T), -7, **i32)
        self.d_parent = torch.full((B, T), -7, **i32)
        self.d_depth = torch.full((B, T), -7, **i32)
        self.d_pos = torch.full((B, T), -7, **i32)
        self.d_mask = torch.zeros(B, T, 2, dtype=torch.int64, device=dev)
        self.d_retrieve = torch.full((B, T, self.max_d + 1), -7, **i32)
        self.d_n_leaves = torch.zeros(B, **i32)
        self.d_n_nodes = torch.zeros(B, **i32)
        self.d_target = torch.zeros(B, T, V, dtype=torch.float32, device=dev)
        self.d_argmax = torch.full((B, T), -7, **i32)
        self.d_path = torch.full((B, self.max_d + 1), -7, **i32)
        self.d_alen = torch.zeros(B, **i32)
        self.d_out = torch.full((B, self.max_d + 1), -7, **i32)
        self.d_q = torch.zeros(B, T, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
        self.d_o = torch.zeros_like(self.d_q)
        self.d_lse = torch.zeros(B, T, w.n_q_heads, dtype=torch.float32, device=dev)
        kv_shape = (B, w.n_kv_heads, self.cap, w.head_dim)
        self.d_k = [torch.zeros(kv_shape, dtype=torch.bfloat16, device=dev) for _ in range(n_layers)]
        self.d_v = [torch.zeros(kv_shape, dtype=torch.bfloat16, device=dev) for _ in range(n_layers)]
        self.k_ptrs = binding.layer_pointer_table(self.d_k)
        self.v_ptrs = binding.layer_pointer_table(self.d_v)
        # host mirrors for the oracle
        self.h_k = [np.zeros(kv_shape, np.uint16) for _ in range(n_layers)]
        self.h_v = [np.zeros(kv_shape, np.uint16) for _ in range(n_layers)]
        self.L = [synth.initial_prefix(w, s) for s in range(B)]
        self.p_agree = [synth.agreement_prob(w, s) for s in range(B)]
        for s in range(B):
            for l in range(n_layers):
                kk, vv = synth.prefix_kv(w, s, l, self.L[s])
                self.h_k[l][s, :, : self.L[s]] = kk
                self.h_v[l][s, :, : self.L[s]] = vv
        for l in range(n_layers):
            self.d_k[l].copy_(u16_to_bf16_cuda(self.h_k[l]))
            self.d_v[l].copy_(u16_to_bf16_cuda(self.h_v[l]))
        self.stats = Stats()
        self.kv_strides = (w.n_kv_heads * self.cap * w.head_dim, self.cap * w.head_dim, w.head_dim)

    # ------------------------------------------------------------------ one step
    def step(self, step: int, attn_layers=(), attn_seqs=None, check_compaction="full"):
        """One whole step with every integer output compared.  check_compaction: "full" downloads the
        caches and compares every slot below the new prefix length, "touched" only the slots the step
        moved (L .. L+a), False nothing."""
        w, B = self.w, self.B
        params = [synth.step_params(w, step, s) for s in range(B)]
        steps_h = np.array([[tt, d, k, self.L[s]] for s, (tt, d, k) in enumerate(params)], np.int32)
        self.d_steps.copy_(torch.from_numpy(steps_h))
        roots = [synth.root_token(w, step, s) for s in range(B)]
        self.d_root.copy_(torch.tensor(roots, dtype=torch.int32))
        drafts = []
        for s, (tt, d, k) in enumerate(params):
            dl = synth.draft_logits(w, step, s, d, k)
            drafts.append(dl)
            self.d_draft[s, :d, :k].copy_(torch.from_numpy(dl))
        V = w.vocab
        binding.resps_tree_expand(
            self.ctx, self.d_steps, B, self.d_draft, self.max_d * self.max_k * V, self.max_k * V, V,
            self.max_d, self.max_k, self.d_root, self.d_tokens, self.d_parent, self.d_depth,
            self.d_pos, self.d_mask, self.d_retrieve, self.d_n_leaves, self.d_n_nodes)
        trees = []
        g_tokens, g_parent = self.d_tokens.cpu().numpy(), self.d_parent.cpu().numpy()
        g_depth, g_pos = self.d_depth.cpu().numpy(), self.d_pos.cpu().numpy()
        g_mask = self.d_mask.cpu().numpy().view(np.uint64)
        g_ret = self.d_retrieve.cpu().numpy()
        g_nl, g_nn = self.d_n_leaves.cpu().numpy(), self.d_n_nodes.cpu().numpy()
        for s, (tt, d, k) in enumerate(params):
            def same_as(t):
                n = t.n_nodes
                return (g_nn[s] == n and g_nl[s] == t.n_leaves
                        and np.array_equal(g_tokens[s, :n], t.tokens)
                        and np.array_equal(g_parent[s, :n], t.parent)
                        and np.array_equal(g_depth[s, :n], t.depth)
                        and np.array_equal(g_pos[s, :n], t.position_ids)
                        and np.array_equal(g_mask[s, :n], t.mask)
                        and np.array_equal(g_ret[s, : t.n_leaves], t.retrieve))
            args = (roots[s], drafts[s], tt, d, k, self.L[s])
            kw = dict(max_tt=self.max_tt, ret_stride=self.max_d + 1)
            t = oracle.tree_expand(*args, tau=TAU, **kw)
            near = t.min_gap < TAU
            self.stats.near_tie_steps += int(near)
            if not same_as(t):
                assert near, (f"tree mismatch at step {step} seq {s} (TT,d,k)={params[s]} "
                              f"min_gap={t.min_gap}: gpu n={g_nn[s]} oracle n={t.n_nodes}")
                # Near tie: the log-sum-exp is summed in another order on the GPU, which may put two
                # candidates whose fp64 scores lie within TAU of each other the other way round.  The
                # GPU's tree must then equal, in every array, the oracle's tree for one of those swaps;
                # the step goes on from that tree.
                for flipped, tv in oracle.tree_expand_swapped(*args, tau=TAU, **kw):
                    if same_as(tv):
                        self.stats.near_tie_swaps.append((step, s, flipped))
                        t = tv
                        break
                else:
                    raise AssertionError(
                        f"tree mismatch at step {step} seq {s} (TT,d,k)={params[s]}: not explained by a swap "
                        f"among the near pairs {t.near_pairs.tolist()} (min_gap={t.min_gap})")
            trees.append(t)
            self.stats.n_nodes.append(t.n_nodes)

        # ---- this step's tree K/V and queries, target logits ---------------------------
        for s, t in enumerate(trees):
            n, L = t.n_nodes, self.L[s]
            for l in range(self.nl):
                kk, vv = synth.tree_kv(w, step, s, l, n)
                self.h_k[l][s, :, L:L + n] = kk
                self.h_v[l][s, :, L:L + n] = vv
                self.d_k[l][s, :, L:L + n].copy_(u16_to_bf16_cuda(kk))
                self.d_v[l][s, :, L:L + n].copy_(u16_to_bf16_cuda(vv))
            tl = synth.target_logits(w, step, s, t.tokens, t.parent, n, self.p_agree[s])
            self.d_target[s, :n].copy_(torch.from_numpy(tl))
            t.target_logits = tl

        # ---- attention -------------------------------------------------------------------
        scale = 1.0 / np.sqrt(w.head_dim)
        for l in attn_layers:
            qs = []
            for s, t in enumerate(trees):
                q = synth.queries(w, step, s, l, t.n_nodes)
                qs.append(q)
                self.d_q[s, : t.n_nodes].copy_(u16_to_bf16_cuda(q))
            self.d_o.fill_(float("nan"))
            binding.resps_tree_attention(
                self.ctx, self.d_steps, self.d_n_nodes, B, self.d_q, self.d_o, self.d_lse,
                self.d_k[l], self.d_v[l], *self.kv_strides, self.cap, self.d_mask, scale)
            g_o = bf16_to_f64(self.d_o)
            g_lse = self.d_lse.cpu().numpy()
            for s, t in enumerate(trees):
                if attn_seqs is not None and s not in attn_seqs:
                    continue
                n = t.n_nodes
                ref, ref_lse = oracle.tree_attention(qs[s], self.h_k[l][s], self.h_v[l][s], self.L[s],
                                                     t.mask, scale, want_lse=True)
                a, r = check_attention(g_o[s, :n], ref)
                np.testing.assert_allclose(g_lse[s, :n], ref_lse, atol=LSE_ABS)
                assert np.isnan(g_o[s, n:]).all(), "rows past n must not be written"
                self.stats.attn_checks += 1
                self.stats.attn_max_abs = max(self.stats.attn_max_abs, a)
                self.stats.attn_max_rel = max(self.stats.attn_max_rel, r)

        # ---- verify / accept -------------------------------------------------------------
        T = self.max_tt
        binding.resps_verify_accept(
            self.ctx, self.d_steps, self.d_n_nodes, B, self.d_target, T * V, V, self.d_tokens,
            self.d_parent, self.d_argmax, self.d_path, self.d_alen, self.d_out, self.d_steps_next)
        g_arg, g_path = self.d_argmax.cpu().numpy(), self.d_path.cpu().numpy()
        g_alen, g_out = self.d_alen.cpu().numpy(), self.d_out.cpu().numpy()
        g_next = self.d_steps_next.cpu().numpy()
        accs = []
        for s, t in enumerate(trees):
            acc = oracle.verify_accept(t.target_logits, t.tokens, t.parent, path_cap=self.max_d + 1)
            accs.append(acc)
            n, a = t.n_nodes, acc.accept_len
            assert np.array_equal(g_arg[s, :n], acc.target_argmax), f"argmax mismatch step {step}"
            assert g_alen[s] == a, f"accept_len {g_alen[s]} != {a} at step {step} seq {s}"
            assert np.array_equal(g_path[s, : a + 1], acc.path) and (g_path[s, a + 1:] == -1).all()
            assert np.array_equal(g_out[s, : a + 1], acc.out_tokens) and (g_out[s, a + 1:] == -1).all()
            assert g_next[s].tolist() == [*steps_h[s, :3], self.L[s] + a + 1]
            self.stats.accept_lens.append(a)

        # ---- compaction ------------------------------------------------------------------
        binding.resps_kv_compact(self.ctx, self.d_steps, B, self.d_path, self.d_alen, self.k_ptrs,
                                 self.v_ptrs, self.nl, *self.kv_strides, self.cap)
        for s, acc in enumerate(accs):
            L = self.L[s]
            for l in range(self.nl):
                oracle.kv_compact(self.h_k[l][s], self.h_v[l][s], L, acc.path)
            self.L[s] = L + acc.accept_len + 1
        if check_compaction == "touched":
            for s, acc in enumerate(accs):
                Ln = self.L[s]
                L0 = Ln - acc.accept_len - 1
                for l in range(self.nl):
                    gk = self.d_k[l][s, :, L0:Ln].contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
                    gv = self.d_v[l][s, :, L0:Ln].contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
                    assert np.array_equal(gk, self.h_k[l][s, :, L0:Ln]), "compacted K differs"
                    assert np.array_equal(gv, self.h_v[l][s, :, L0:Ln]), "compacted V differs"
        elif check_compaction:
            for l in range(self.nl):
                gk = self.d_k[l].view(torch.int16).cpu().numpy().view(np.uint16)
                gv = self.d_v[l].view(torch.int16).cpu().numpy().view(np.uint16)
                for s in range(B):
                    Ln = self.L[s]
                    assert np.array_equal(gk[s, :, :Ln], self.h_k[l][s, :, :Ln]), "compacted K differs"
                    assert np.array_equal(gv[s, :, :Ln], self.h_v[l][s, :, :Ln]), "compacted V differs"
        assert self.ctx.status() == 0
        self.stats.steps += 1

    def close(self):
        torch.cuda.synchronize()
        self.ctx.close()
