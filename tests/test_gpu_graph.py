"""One CUDA graph of a whole step (expand, attention, verify, compaction), captured once and replayed
while (TT, d, k), the prefix lengths and all inputs change in device memory between replays: nothing
about a launch may depend on the step parameters.  Every replay is compared with the oracle."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_one_captured_step_graph_serves_changing_tree_shapes():
    from harness import Runner, check_attention, u16_to_bf16_cuda, bf16_to_f64, TAU
    from paper_2601_12212_b200 import binding, synth
    import oracle

    w = synth.Workload(7, "graph-replay", 2, 8, 2, 128, 5000, 1, 1536, 64, "gumbel_peaked", "grid", 80, 8, 12,
                       (300, 900), (0.6, 0.9), hold=1)
    r = Runner(w, n_layers=1)
    B, V, T = r.B, w.vocab, r.max_tt
    scale = 1.0 / np.sqrt(w.head_dim)
    stream = torch.cuda.Stream()

    def launch_step():
        binding.resps_tree_expand(
            r.ctx, r.d_steps, B, r.d_draft, r.max_d * r.max_k * V, r.max_k * V, V, r.max_d, r.max_k, r.d_root,
            r.d_tokens, r.d_parent, r.d_depth, r.d_pos, r.d_mask, r.d_retrieve, r.d_n_leaves, r.d_n_nodes,
            stream=stream)
        binding.resps_tree_attention(r.ctx, r.d_steps, r.d_n_nodes, B, r.d_q, r.d_o, r.d_lse, r.d_k[0], r.d_v[0],
                                     *r.kv_strides, r.cap, r.d_mask, scale, stream=stream)
        binding.resps_verify_accept(r.ctx, r.d_steps, r.d_n_nodes, B, r.d_target, T * V, V, r.d_tokens, r.d_parent,
                                    r.d_argmax, r.d_path, r.d_alen, r.d_out, r.d_steps_next, stream=stream)
        binding.resps_kv_compact(r.ctx, r.d_steps, B, r.d_path, r.d_alen, r.k_ptrs, r.v_ptrs, 1, *r.kv_strides,
                                 r.cap, stream=stream)

    graph = None
    shapes = set()
    for step in range(7):
        params = [synth.step_params(w, step, s) for s in range(B)]
        shapes.update(params)
        steps_h = np.array([[tt, d, k, r.L[s]] for s, (tt, d, k) in enumerate(params)], np.int32)
        roots = [synth.root_token(w, step, s) for s in range(B)]
        trees, qs = [], []
        r.d_steps.copy_(torch.from_numpy(steps_h))
        r.d_root.copy_(torch.tensor(roots, dtype=torch.int32))
        for s, (tt, d, k) in enumerate(params):
            dl = synth.draft_logits(w, step, s, d, k)
            r.d_draft[s, :d, :k].copy_(torch.from_numpy(dl))
            t = oracle.tree_expand(roots[s], dl, tt, d, k, r.L[s], max_tt=T, ret_stride=r.max_d + 1)
            assert t.min_gap >= TAU, "the seeded inputs of this test have no near ties"
            trees.append(t)
            n, L = t.n_nodes, r.L[s]
            kk, vv = synth.tree_kv(w, step, s, 0, n)
            r.h_k[0][s, :, L:L + n] = kk
            r.h_v[0][s, :, L:L + n] = vv
            r.d_k[0][s, :, L:L + n].copy_(u16_to_bf16_cuda(kk))
            r.d_v[0][s, :, L:L + n].copy_(u16_to_bf16_cuda(vv))
            t.target_logits = synth.target_logits(w, step, s, t.tokens, t.parent, n, r.p_agree[s])
            r.d_target[s, :n].copy_(torch.from_numpy(t.target_logits))
            q = synth.queries(w, step, s, 0, n)
            qs.append(q)
            r.d_q[s, :n].copy_(u16_to_bf16_cuda(q))
        r.d_o.fill_(float("nan"))
        torch.cuda.synchronize()
        if graph is None:
            with torch.cuda.stream(stream):
                launch_step()  # a first, plain pass loads the kernels; its results are overwritten below
            torch.cuda.synchronize()
            # undo what the plain pass did to the cache, then capture the same calls
            for l in range(1):
                r.d_k[l].copy_(u16_to_bf16_cuda(r.h_k[l]))
                r.d_v[l].copy_(u16_to_bf16_cuda(r.h_v[l]))
            r.d_o.fill_(float("nan"))
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                launch_step()
        graph.replay()
        torch.cuda.synchronize()
        assert r.ctx.status() == 0

        g_tokens, g_parent = r.d_tokens.cpu().numpy(), r.d_parent.cpu().numpy()
        g_mask = r.d_mask.cpu().numpy().view(np.uint64)
        g_ret, g_nn, g_nl = r.d_retrieve.cpu().numpy(), r.d_n_nodes.cpu().numpy(), r.d_n_leaves.cpu().numpy()
        g_o, g_arg = bf16_to_f64(r.d_o), r.d_argmax.cpu().numpy()
        g_path, g_alen, g_out = r.d_path.cpu().numpy(), r.d_alen.cpu().numpy(), r.d_out.cpu().numpy()
        g_next = r.d_steps_next.cpu().numpy()
        for s, t in enumerate(trees):
            n = t.n_nodes
            assert g_nn[s] == n and g_nl[s] == t.n_leaves
            assert np.array_equal(g_tokens[s, :n], t.tokens) and np.array_equal(g_parent[s, :n], t.parent)
            assert np.array_equal(g_mask[s, :n], t.mask) and np.array_equal(g_ret[s, : t.n_leaves], t.retrieve)
            ref = oracle.tree_attention(qs[s], r.h_k[0][s], r.h_v[0][s], r.L[s], t.mask, scale)
            check_attention(g_o[s, :n], ref)
            assert np.isnan(g_o[s, n:]).all()
            acc = oracle.verify_accept(t.target_logits, t.tokens, t.parent, path_cap=r.max_d + 1)
            a = acc.accept_len
            assert np.array_equal(g_arg[s, :n], acc.target_argmax) and g_alen[s] == a
            assert np.array_equal(g_path[s, : a + 1], acc.path) and np.array_equal(g_out[s, : a + 1], acc.out_tokens)
            assert g_next[s].tolist() == [*steps_h[s, :3], r.L[s] + a + 1]
            oracle.kv_compact(r.h_k[0][s], r.h_v[0][s], r.L[s], acc.path)
            r.L[s] += a + 1
        gk = r.d_k[0].view(torch.int16).cpu().numpy().view(np.uint16)
        gv = r.d_v[0].view(torch.int16).cpu().numpy().view(np.uint16)
        for s in range(B):
            assert np.array_equal(gk[s, :, : r.L[s]], r.h_k[0][s, :, : r.L[s]])
            assert np.array_equal(gv[s, :, : r.L[s]], r.h_v[0][s, :, : r.L[s]])
    assert len(shapes) >= 4  # the tree shape really changed under the one captured graph
    r.close()
