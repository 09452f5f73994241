"""Vocabulary sharding: four "ranks" (here: four contexts on one GPU, one after the other -- a call on
this pool gets a single GPU) each scan their own columns of every logits row; the merged results must be
the tree and the acceptance of the unsharded calls and of the oracle."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("index,steps_n", [(2, 2), (1, 4)])
def test_sharded_vocabulary_equals_the_unsharded_step(index, steps_n):
    import oracle
    from harness import Runner, TAU
    from paper_2601_12212_b200 import binding, synth
    w = synth.WORKLOADS[index]
    r = Runner(w, n_layers=1)                      # the unsharded context and all buffers
    B, V, T = r.B, w.vocab, r.max_tt
    P = 4
    cols = binding.shard_columns(V, P)
    assert sum(wd for _, wd in cols) == V and all(off % 4 == 0 for off, _ in cols)
    ctxs = [binding.Context(w.n_q_heads, w.n_kv_heads, w.head_dim, wd, max_batch=B, max_tt=T, max_k=r.max_k,
                            max_depth=r.max_d) for _, wd in cols]
    rows = int(binding.load().resps_scan_rows(ctxs[0].handle))
    i32 = dict(dtype=torch.int32, device="cuda")
    d_off = torch.tensor([off for off, _ in cols], **i32)
    for step in range(steps_n):
        params = [synth.step_params(w, step, s) for s in range(B)]
        steps_h = np.array([[tt, d, k, r.L[s]] for s, (tt, d, k) in enumerate(params)], np.int32)
        r.d_steps.copy_(torch.from_numpy(steps_h))
        roots = [synth.root_token(w, step, s) for s in range(B)]
        r.d_root.copy_(torch.tensor(roots, dtype=torch.int32))
        drafts = [synth.draft_logits(w, step, s, d, k) for s, (tt, d, k) in enumerate(params)]
        for s, (tt, d, k) in enumerate(params):
            r.d_draft[s, :d, :k].copy_(torch.from_numpy(drafts[s]))
        ldb, ldl = r.max_d * r.max_k * V, r.max_k * V
        flat = r.d_draft.view(-1)
        # ---- every rank scans its columns; "all-gather" = stacking the ranks' small results -------------
        vals, ids, lses = [], [], []
        for (off, wd), ctx in zip(cols, ctxs):
            pv = torch.zeros(B, rows, r.max_k, device="cuda")
            pi = torch.zeros(B, rows, r.max_k, **i32)
            pl = torch.zeros(B, rows, dtype=torch.float64, device="cuda")
            binding.resps_row_scan_shard(ctx, r.d_steps, B, flat[off:], ldb, ldl, V, r.max_d, r.max_k, pv, pi, pl)
            assert ctx.status() == 0
            vals.append(pv), ids.append(pi), lses.append(pl)
        all_val, all_id, all_lse = torch.stack(vals), torch.stack(ids), torch.stack(lses)
        outs = [torch.full((B, T), -7, **i32) for _ in range(4)] + \
               [torch.zeros(B, T, 2, dtype=torch.int64, device="cuda"), torch.full((B, T, r.max_d + 1), -7, **i32),
                torch.zeros(B, **i32), torch.zeros(B, **i32)]
        binding.resps_tree_expand_merge(ctxs[1], r.d_steps, B, r.max_d, r.max_k, P, all_val, all_id, all_lse, d_off,
                                        r.d_root, *outs)
        assert ctxs[1].status() == 0
        binding.resps_tree_expand(r.ctx, r.d_steps, B, r.d_draft, ldb, ldl, V, r.max_d, r.max_k, r.d_root, r.d_tokens,
                                  r.d_parent, r.d_depth, r.d_pos, r.d_mask, r.d_retrieve, r.d_n_leaves, r.d_n_nodes)
        whole = [r.d_tokens, r.d_parent, r.d_depth, r.d_pos, r.d_mask, r.d_retrieve, r.d_n_leaves, r.d_n_nodes]
        trees = []
        for s, (tt, d, k) in enumerate(params):
            t = oracle.tree_expand(roots[s], drafts[s], tt, d, k, r.L[s], max_tt=T, ret_stride=r.max_d + 1, tau=TAU)
            assert t.min_gap >= TAU
            trees.append(t)
            n = t.n_nodes
            assert int(outs[7][s]) == n and np.array_equal(outs[0][s, :n].cpu().numpy(), t.tokens)
            assert np.array_equal(outs[1][s, :n].cpu().numpy(), t.parent)
            assert np.array_equal(outs[4][s, :n].cpu().numpy().view(np.uint64), t.mask)
            for i_out in range(5):                                    # tokens, parent, depth, position ids, mask
                assert torch.equal(outs[i_out][s, :n], whole[i_out][s, :n])
            assert int(outs[6][s]) == int(whole[6][s]) == t.n_leaves and int(whole[7][s]) == n
            assert torch.equal(outs[5][s, : t.n_leaves], whole[5][s, : t.n_leaves])
            tl = synth.target_logits(w, step, s, t.tokens, t.parent, n, r.p_agree[s])
            tl[: n, cols[2][0] + 3] = tl[: n, 5]                       # a tie across two shards: the lower id wins
            r.d_target[s, :n].copy_(torch.from_numpy(tl))
            t.target_logits = tl
        # ---- verification --------------------------------------------------------------------------------
        tflat = r.d_target.view(-1)
        keys = []
        for (off, wd), ctx in zip(cols, ctxs):
            pk = torch.zeros(B, T, dtype=torch.int64, device="cuda")
            binding.resps_target_argmax_shard(ctx, outs[7], B, tflat[off:], T * V, V, pk)
            keys.append(pk)
        amax = torch.full((B, T), -7, **i32)
        path = torch.full((B, r.max_d + 1), -7, **i32)
        alen = torch.zeros(B, **i32)
        otok = torch.full((B, r.max_d + 1), -7, **i32)
        binding.resps_verify_accept_merge(ctxs[3], r.d_steps, outs[7], B, P, torch.stack(keys), d_off, outs[0], outs[1],
                                          amax, path, alen, otok, r.d_steps_next)
        assert ctxs[3].status() == 0
        for s, t in enumerate(trees):
            acc = oracle.verify_accept(t.target_logits, t.tokens, t.parent, path_cap=r.max_d + 1)
            a, n = acc.accept_len, t.n_nodes
            assert np.array_equal(amax[s, :n].cpu().numpy(), acc.target_argmax)
            assert int(alen[s]) == a and np.array_equal(path[s, : a + 1].cpu().numpy(), acc.path)
            assert np.array_equal(otok[s, : a + 1].cpu().numpy(), acc.out_tokens)
            assert r.d_steps_next[s].tolist() == [*steps_h[s, :3], r.L[s] + a + 1]
    for c in ctxs:
        c.close()
    r.close()
