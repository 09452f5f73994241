"""The level form of the tree expansion (begin / one call per level / finish), as a draft model that runs
between levels would drive it: every level's frontier equals the oracle's, the finished tree equals both
the oracle's and the whole-step call's, and the frontier masks drive resps_tree_attention for the
draft-side pass over prefix + draft nodes."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_level_form_equals_the_whole_step_form_and_the_oracle():
    import oracle
    from harness import TAU
    from paper_2601_12212_b200 import binding, synth
    w = synth.Workload(10, "level-form", 3, 8, 2, 128, 5000, 1, 1536, 64, "gumbel_peaked", "grid", 80, 8, 12,
                       (300, 900), (0.6, 0.9), hold=1)
    B, V, T, MK, MD = 3, w.vocab, 80, 12, 8
    ctx = binding.Context(w.n_q_heads, w.n_kv_heads, w.head_dim, V, max_batch=B, max_tt=T, max_k=MK, max_depth=MD)
    i32 = dict(dtype=torch.int32, device="cuda")
    for step in range(4):
        params = [synth.step_params(w, step, s) for s in range(B)]
        Ls = [100 + 7 * s for s in range(B)]
        steps = torch.tensor([[*p, L] for p, L in zip(params, Ls)], **i32)
        roots = [synth.root_token(w, step, s) for s in range(B)]
        d_root = torch.tensor(roots, **i32)
        drafts = [synth.draft_logits(w, step, s, d, k) for s, (tt, d, k) in enumerate(params)]
        d_all = torch.zeros(B, MD, MK, V, device="cuda")
        for s, (tt, d, k) in enumerate(params):
            d_all[s, :d, :k].copy_(torch.from_numpy(drafts[s]))
        trees = [oracle.tree_expand(roots[s], drafts[s], tt, d, k, Ls[s], max_tt=T, ret_stride=MD + 1, tau=TAU)
                 for s, (tt, d, k) in enumerate(params)]
        assert all(t.min_gap >= TAU for t in trees)

        def outputs():
            return ([torch.full((B, T), -7, **i32) for _ in range(4)] +
                    [torch.zeros(B, T, 2, dtype=torch.int64, device="cuda"), torch.full((B, T, MD + 1), -7, **i32),
                     torch.zeros(B, **i32), torch.zeros(B, **i32)])

        # ---- level by level ---------------------------------------------------------------------------
        binding.resps_tree_expand_begin(ctx, steps, B, MK)
        f_tok, f_par, f_pos, f_idx = (torch.full((B, MK), -7, **i32) for _ in range(4))
        f_mask = torch.zeros(B, MK, 2, dtype=torch.int64, device="cuda")
        f_score = torch.zeros(B, MK, dtype=torch.float64, device="cuda")
        for j in range(max(d for _, d, _ in params)):
            rows = d_all[:, j].contiguous()                               # what the draft model hands over: [B][MK][V]
            binding.resps_tree_expand_level(ctx, steps, B, j, rows, MK * V, V, f_tok, f_par, f_pos, f_idx, f_mask, f_score)
            g = [x.cpu().numpy() for x in (f_tok, f_par, f_pos, f_idx)]
            g_mask = f_mask.cpu().numpy().view(np.uint64)
            g_score = f_score.cpu().numpy()
            for s, (tt, d, k) in enumerate(params):
                if j >= d:
                    continue
                want = trees[s].level_frontier(j, k, Ls[s])
                for got, name in zip(g, ("tokens", "parent_slot", "position_ids", "node_index")):
                    assert np.array_equal(got[s, :k], want[name]), (step, s, j, name)
                if 1 + (j + 1) * k <= 128:
                    assert np.array_equal(g_mask[s, :k], want["mask"])
                np.testing.assert_allclose(g_score[s, :k], want["score"], atol=1e-5)
        level_out = outputs()
        binding.resps_tree_expand_finish(ctx, steps, B, d_root, *level_out)
        status = ctx.status()
        # sequences whose d is below the deepest one were "given" more levels than they use: no flag for that
        assert status == 0
        # ---- the whole step at once -----------------------------------------------------------------------
        whole_out = outputs()
        binding.resps_tree_expand(ctx, steps, B, d_all, MD * MK * V, MK * V, V, MD, MK, d_root, *whole_out)
        assert ctx.status() == 0
        for a, b in zip(level_out, whole_out):
            assert torch.equal(a, b)
        tok, par = level_out[0].cpu().numpy(), level_out[1].cpu().numpy()
        nn = level_out[7].cpu().numpy()
        for s, t in enumerate(trees):
            assert nn[s] == t.n_nodes and np.array_equal(tok[s, : t.n_nodes], t.tokens)
            assert np.array_equal(par[s, : t.n_nodes], t.parent)
    # levels out of order are refused
    binding.resps_tree_expand_begin(ctx, steps, B, MK)
    with pytest.raises(binding.RespsError):
        binding.resps_tree_expand_level(ctx, steps, B, 1, d_all[:, 1].contiguous(), MK * V, V, f_tok, f_par, f_pos,
                                        f_idx, f_mask, None)
    ctx.close()


def test_draft_side_attention_over_the_frontier_masks():
    """The draft model's pass for level j: queries are the draft nodes so far (root, then the frontiers of
    levels 0..j, k each), every node seeing the prefix and its ancestors.  The masks come from the level
    calls; the attention is the same kernel as on the target side."""
    import oracle
    from harness import check_attention, u16_to_bf16_cuda, bf16_to_f64
    from paper_2601_12212_b200 import binding, synth
    rng = np.random.default_rng(2)
    V, k, d, L, Hq, Hkv, D, cap = 3000, 6, 4, 333, 8, 2, 128, 512
    T = 1 + d * k
    ctx = binding.Context(Hq, Hkv, D, V, max_batch=1, max_tt=T, max_k=k, max_depth=d)
    i32 = dict(dtype=torch.int32, device="cuda")
    logits = rng.normal(size=(d, k, V)).astype(np.float32) * 2
    steps = torch.tensor([[T, d, k, L]], **i32)
    f = [torch.zeros(1, k, **i32) for _ in range(4)]
    f_mask = torch.zeros(1, k, 2, dtype=torch.int64, device="cuda")
    masks = np.zeros((1, T, 2), np.uint64)
    masks[0, 0, 0] = 1
    q = synth.to_bf16_bits(rng.normal(size=(1, T, Hq, D)).astype(np.float32).ravel()).reshape(1, T, Hq, D)
    kc = synth.to_bf16_bits(rng.normal(size=(1, Hkv, cap, D)).astype(np.float32).ravel()).reshape(1, Hkv, cap, D)
    vc = synth.to_bf16_bits(rng.normal(size=(1, Hkv, cap, D)).astype(np.float32).ravel()).reshape(1, Hkv, cap, D)
    dq, dk, dv = u16_to_bf16_cuda(q), u16_to_bf16_cuda(kc), u16_to_bf16_cuda(vc)
    do = torch.zeros_like(dq)
    binding.resps_tree_expand_begin(ctx, steps, 1, k)
    for j in range(d):
        rows = torch.from_numpy(logits[j][None]).cuda()
        binding.resps_tree_expand_level(ctx, steps, 1, j, rows, k * V, V, *f, f_mask, None)
        n = 1 + (j + 1) * k
        masks[0, 1 + j * k: n] = f_mask.cpu().numpy().view(np.uint64)[0]
        nn = torch.tensor([n], **i32)
        dm = torch.from_numpy(masks.view(np.int64)).cuda()
        binding.resps_tree_attention(ctx, steps, nn, 1, dq, do, None, dk, dv, Hkv * cap * D, cap * D, D, cap, dm,
                                     1 / np.sqrt(D))
        assert ctx.status() == 0
        ref = oracle.tree_attention(q[0, :n], kc[0], vc[0], L, masks[0, :n], 1 / np.sqrt(D))
        check_attention(bf16_to_f64(do)[0, 1 + j * k: n], ref[1 + j * k: n])    # the new frontier's rows
    ctx.close()
