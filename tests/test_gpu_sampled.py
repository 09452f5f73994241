"""Acceptance under sampling (temperature > 0) on the GPU against the fp64 oracle, through the C-ABI.
Every decision of the walk (accept or reject a child, which token is drawn) must be the oracle's
whenever the oracle's margin for it exceeds 1e-9 (both sides compute in fp64 and differ only in the
order of their sums); accepted path, length and tokens are then compared bit for bit."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

MARGIN = 1e-9


def _run(w, temperature, steps, seed):
    import oracle
    from harness import Runner, TAU
    from paper_2601_12212_b200 import binding, synth
    r = Runner(w, n_layers=1)
    B, V, T = r.B, w.vocab, r.max_tt
    cap = r.max_d + 1
    rng = np.random.default_rng(seed)
    d_ua = torch.zeros(B, cap, r.max_k, dtype=torch.float64, device="cuda")
    d_us = torch.zeros(B, cap, dtype=torch.float64, device="cuda")
    lens, checked, rejected_then_accepted = [], 0, 0
    for step in range(steps):
        params = [synth.step_params(w, step, s) for s in range(B)]
        steps_h = np.array([[tt, d, k, r.L[s]] for s, (tt, d, k) in enumerate(params)], np.int32)
        r.d_steps.copy_(torch.from_numpy(steps_h))
        roots = [synth.root_token(w, step, s) for s in range(B)]
        r.d_root.copy_(torch.tensor(roots, dtype=torch.int32))
        drafts = []
        for s, (tt, d, k) in enumerate(params):
            dl = synth.draft_logits(w, step, s, d, k)
            drafts.append(dl)
            r.d_draft[s, :d, :k].copy_(torch.from_numpy(dl))
        binding.resps_tree_expand(
            r.ctx, r.d_steps, B, r.d_draft, r.max_d * r.max_k * V, r.max_k * V, V, r.max_d, r.max_k, r.d_root,
            r.d_tokens, r.d_parent, r.d_depth, r.d_pos, r.d_mask, r.d_retrieve, r.d_n_leaves, r.d_n_nodes)
        trees = []
        g_tokens, g_parent = r.d_tokens.cpu().numpy(), r.d_parent.cpu().numpy()
        for s, (tt, d, k) in enumerate(params):
            t = oracle.tree_expand(roots[s], drafts[s], tt, d, k, r.L[s], max_tt=T, ret_stride=cap, tau=TAU)
            assert t.min_gap >= TAU
            assert np.array_equal(g_tokens[s, : t.n_nodes], t.tokens) and np.array_equal(g_parent[s, : t.n_nodes], t.parent)
            trees.append(t)
            tl = synth.target_logits(w, step, s, t.tokens, t.parent, t.n_nodes, r.p_agree[s])
            r.d_target[s, : t.n_nodes].copy_(torch.from_numpy(tl))
            t.target_logits = tl
        ua = rng.uniform(size=(B, cap, r.max_k))
        us = rng.uniform(size=(B, cap))
        d_ua.copy_(torch.from_numpy(ua))
        d_us.copy_(torch.from_numpy(us))
        binding.resps_verify_accept_sampled(
            r.ctx, r.d_steps, r.d_n_nodes, B, r.d_target, T * V, V, r.d_draft, r.max_d * r.max_k * V, r.max_k * V, V,
            temperature, r.d_tokens, r.d_parent, d_ua, d_us, r.d_path, r.d_alen, r.d_out, r.d_steps_next)
        assert r.ctx.status() == 0
        g_path, g_alen, g_out = r.d_path.cpu().numpy(), r.d_alen.cpu().numpy(), r.d_out.cpu().numpy()
        g_next = r.d_steps_next.cpu().numpy()
        for s, t in enumerate(trees):
            tt, d, k = params[s]
            rows = np.zeros((r.max_d * 32, V), np.float32)      # row index = level * 32 + slot, as the library keeps it
            for lvl in range(d):
                rows[lvl * 32: lvl * 32 + k] = drafts[s][lvl]
            node_row = t.node_rows(d, k, 32)
            o = oracle.verify_accept_sampled(t.target_logits, rows, node_row, t.tokens, t.parent, temperature,
                                             ua[s], us[s], path_cap=cap)
            lens.append(o.accept_len)
            if o.min_margin <= MARGIN:
                continue                                         # a decision on a knife's edge: either answer is right
            checked += 1
            a = o.accept_len
            assert g_alen[s] == a, f"step {step} seq {s}: accept_len {g_alen[s]} != {a} (margin {o.min_margin})"
            assert np.array_equal(g_path[s, : a + 1], o.path) and (g_path[s, a + 1:] == -1).all()
            assert np.array_equal(g_out[s, : a + 1], o.out_tokens) and (g_out[s, a + 1:] == -1).all()
            assert g_next[s].tolist() == [*steps_h[s, :3], r.L[s] + a + 1]
    r.close()
    return lens, checked


def test_sampled_acceptance_tiny_diffuse_logits():
    """N(0, 2) logits at T = 1: probabilities are spread out, children are often rejected and later
    siblings accepted against residuals."""
    from paper_2601_12212_b200 import synth
    lens, checked = _run(synth.WORKLOADS[1], 1.0, 40, seed=1)
    assert checked >= 38 and max(lens) >= 1 and min(lens) == 0


@pytest.mark.parametrize("temperature", [0.7, 1.5])
def test_sampled_acceptance_batch_of_varying_trees(temperature):
    from paper_2601_12212_b200 import synth
    w = synth.Workload(9, "sampled", 3, 8, 2, 128, 5000, 1, 1536, 64, "gumbel_peaked", "grid", 80, 8, 12,
                       (300, 900), (0.6, 0.9), hold=1)
    lens, checked = _run(w, temperature, 10, seed=int(temperature * 10))
    assert checked >= 28 and max(lens) >= 2


def test_sampled_acceptance_llama8b_shape():
    """Vocabulary 128256, TT = 60: the sums run over 10^5 terms in eight CTAs."""
    from paper_2601_12212_b200 import synth
    lens, checked = _run(synth.WORKLOADS[2], 1.0, 3, seed=3)
    assert checked >= 3


def test_sampled_acceptance_wide_vocabulary():
    """Vocabulary 200 000: a CTA's slice of two rows no longer fits the staging area in shared memory, so
    the rows are read in place (the other path of the kernel); two sequences, small trees."""
    from paper_2601_12212_b200 import synth
    w = synth.Workload(10, "sampled-wide", 2, 8, 2, 128, 200000, 1, 1024, 16, "gumbel_peaked", "fixed", 12, 3, 4,
                       (100, 300), 0.7)
    lens, checked = _run(w, 1.0, 3, seed=5)
    assert checked >= 5
