"""The step loop advances on the device: one CUDA graph of a whole step is captured once and replayed
18 times while the host never writes the prefix lengths.  resps_verify_accept writes the advanced
step array over the one it read (d_steps_next aliases d_steps) and resps_kv_compact is told so
(steps_advanced = 1).  The host only refreshes inputs a model would produce (logits, Q, the tree
tokens' K/V) and the per-step (TT, d, k), through a device-side copy that is part of the graph.
Every replay is compared with the oracle, which keeps its own prefix lengths."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_device_resident_loop():
    from harness import Runner, check_attention, u16_to_bf16_cuda, bf16_to_f64, TAU
    from paper_2601_12212_b200 import binding, synth
    import oracle

    w = synth.Workload(8, "device-loop", 2, 8, 2, 128, 5000, 1, 1536, 64, "gumbel_peaked", "grid", 80, 8, 12,
                       (300, 900), (0.6, 0.9), hold=2)
    r = Runner(w, n_layers=1)
    B, V, T = r.B, w.vocab, r.max_tt
    scale = 1.0 / np.sqrt(w.head_dim)
    stream = torch.cuda.Stream()
    d_params = torch.zeros(B, 3, dtype=torch.int32, device="cuda")   # this step's (TT, d, k), written by the host
    # the prefix lengths are written once, before the first step
    r.d_steps.copy_(torch.tensor([[0, 0, 0, r.L[s]] for s in range(B)], dtype=torch.int32))

    def launch_step():
        r.d_steps[:, :3].copy_(d_params)     # a device-side copy inside the graph; column 3 is never touched
        binding.resps_tree_expand(
            r.ctx, r.d_steps, B, r.d_draft, r.max_d * r.max_k * V, r.max_k * V, V, r.max_d, r.max_k, r.d_root,
            r.d_tokens, r.d_parent, r.d_depth, r.d_pos, r.d_mask, r.d_retrieve, r.d_n_leaves, r.d_n_nodes,
            stream=stream)
        binding.resps_tree_attention(r.ctx, r.d_steps, r.d_n_nodes, B, r.d_q, r.d_o, r.d_lse, r.d_k[0], r.d_v[0],
                                     *r.kv_strides, r.cap, r.d_mask, scale, stream=stream)
        binding.resps_verify_accept(r.ctx, r.d_steps, r.d_n_nodes, B, r.d_target, T * V, V, r.d_tokens, r.d_parent,
                                    r.d_argmax, r.d_path, r.d_alen, r.d_out, r.d_steps, stream=stream)   # in place
        binding.resps_kv_compact(r.ctx, r.d_steps, B, r.d_path, r.d_alen, r.k_ptrs, r.v_ptrs, 1, *r.kv_strides,
                                 r.cap, steps_advanced=True, stream=stream)

    graph = None
    n_steps = 18
    for step in range(n_steps):
        params = [synth.step_params(w, step, s) for s in range(B)]
        roots = [synth.root_token(w, step, s) for s in range(B)]
        trees, qs = [], []
        d_params.copy_(torch.tensor(params, dtype=torch.int32))
        r.d_root.copy_(torch.tensor(roots, dtype=torch.int32))
        for s, (tt, d, k) in enumerate(params):
            dl = synth.draft_logits(w, step, s, d, k)
            r.d_draft[s, :d, :k].copy_(torch.from_numpy(dl))
            t = oracle.tree_expand(roots[s], dl, tt, d, k, r.L[s], max_tt=T, ret_stride=r.max_d + 1, tau=TAU)
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
            # a first, plain pass loads the kernels; undo what it did to the cache and the prefix, then capture
            keep = r.d_steps.clone()
            with torch.cuda.stream(stream):
                launch_step()
            torch.cuda.synchronize()
            r.d_steps.copy_(keep)
            r.d_k[0].copy_(u16_to_bf16_cuda(r.h_k[0]))
            r.d_v[0].copy_(u16_to_bf16_cuda(r.h_v[0]))
            r.d_o.fill_(float("nan"))
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                launch_step()
        graph.replay()
        torch.cuda.synchronize()
        assert r.ctx.status() == 0

        g_tokens, g_parent, g_pos = r.d_tokens.cpu().numpy(), r.d_parent.cpu().numpy(), r.d_pos.cpu().numpy()
        g_mask = r.d_mask.cpu().numpy().view(np.uint64)
        g_nn = r.d_n_nodes.cpu().numpy()
        g_o, g_arg = bf16_to_f64(r.d_o), r.d_argmax.cpu().numpy()
        g_path, g_alen, g_out = r.d_path.cpu().numpy(), r.d_alen.cpu().numpy(), r.d_out.cpu().numpy()
        g_steps = r.d_steps.cpu().numpy()
        for s, t in enumerate(trees):
            n = t.n_nodes
            assert g_nn[s] == n
            assert np.array_equal(g_tokens[s, :n], t.tokens) and np.array_equal(g_parent[s, :n], t.parent)
            assert np.array_equal(g_pos[s, :n], t.position_ids)      # L + depth, with the device's own L
            assert np.array_equal(g_mask[s, :n], t.mask)
            ref = oracle.tree_attention(qs[s], r.h_k[0][s], r.h_v[0][s], r.L[s], t.mask, scale)
            check_attention(g_o[s, :n], ref)
            acc = oracle.verify_accept(t.target_logits, t.tokens, t.parent, path_cap=r.max_d + 1)
            a = acc.accept_len
            assert np.array_equal(g_arg[s, :n], acc.target_argmax) and g_alen[s] == a
            assert np.array_equal(g_path[s, : a + 1], acc.path) and np.array_equal(g_out[s, : a + 1], acc.out_tokens)
            oracle.kv_compact(r.h_k[0][s], r.h_v[0][s], r.L[s], acc.path)
            r.L[s] += a + 1
            assert g_steps[s].tolist() == [*params[s], r.L[s]]       # advanced in place, on the device
        gk = r.d_k[0].view(torch.int16).cpu().numpy().view(np.uint16)
        gv = r.d_v[0].view(torch.int16).cpu().numpy().view(np.uint16)
        for s in range(B):
            assert np.array_equal(gk[s, :, : r.L[s]], r.h_k[0][s, :, : r.L[s]])
            assert np.array_equal(gv[s, :, : r.L[s]], r.h_v[0][s, :, : r.L[s]])
    assert min(r.L) > 300 + n_steps           # every sequence moved on every step
    r.close()
