"""resps_target_argmax_static: the arg-max step for callers that may not allocate device memory
(a process whose GPU memory was handed to another allocator at start-up, or code that only runs
where cudaMalloc is forbidden).  It needs no context; its scratch is a fixed array inside the
library.  Checked here through the C-ABI against what resps_verify_accept writes, bit for bit,
on two calls in a row (the second call finds the array as the first one left it), and -- since
both entry points run the same kernel -- against the CPU oracle's arg-max of the same rows.
The shapes cover one piece per row, many pieces per row, rows of odd length on the scalar path
with several pieces, and a vocabulary so large that the pieces are made longer than 8192.

Collected last on purpose: a run that stops at the first failure has then run every other test."""
import ctypes

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _reference_argmax(binding, torch, logits, n_nodes, T, V):
    """d_target_argmax as the context-owning entry point computes it."""
    B = logits.shape[0]
    ctx = binding.Context(4, 1, 64, V, max_batch=B, max_tt=T, max_k=4, max_depth=4)
    i32 = dict(dtype=torch.int32, device="cuda")
    steps = torch.tensor([[T, 1, 1, 0]] * B, **i32)
    tokens = torch.zeros(B, T, **i32)
    parent = torch.full((B, T), -1, **i32)
    out = torch.full((B, T), -7, **i32)
    path = torch.zeros(B, 5, **i32)
    alen = torch.zeros(B, **i32)
    otok = torch.zeros(B, 5, **i32)
    binding.resps_verify_accept(ctx, steps, n_nodes, B, logits, T * V, V, tokens, parent, out, path, alen, otok)
    torch.cuda.synchronize()
    ctx.close()
    return out.cpu().numpy()


@pytest.mark.parametrize("B,T,V", [(2, 60, 128256), (3, 17, 1001), (2, 5, 20001), (1, 2, 600001)])
def test_static_argmax_matches_verify_accept_twice_in_a_row(B, T, V):
    import torch
    import oracle
    from paper_2601_12212_b200 import binding
    g = torch.Generator(device="cuda")
    g.manual_seed(B * 1000 + T)
    n_nodes = torch.tensor([T, max(1, T // 2), 1][:B], dtype=torch.int32, device="cuda")
    for call in range(2):
        logits = torch.randn(B, T, V, generator=g, device="cuda")
        logits[:, :, V // 3] = logits[:, :, 7]            # ties: the lower id must win
        logits[:, ::2, 7] = 50.0                          # ... also where the tied value is the maximum,
        logits[:, ::2, V // 3] = 50.0                     # in different pieces of the row
        want = _reference_argmax(binding, torch, logits, n_nodes, T, V)
        got = torch.full((B, T), -7, dtype=torch.int32, device="cuda")
        binding.resps_target_argmax_static(n_nodes, B, T, V, logits, T * V, V, got)
        torch.cuda.synchronize()
        got = got.cpu().numpy()
        host = logits.cpu().numpy()
        for b in range(B):
            n = int(n_nodes[b])
            assert np.array_equal(got[b, :n], want[b, :n]), f"call {call}, sequence {b}"
            assert (got[b, n:] == -7).all(), "entries past n_nodes must stay untouched"
            ref = oracle.verify_accept(host[b, :n], np.zeros(n, np.int32), np.full(n, -1, np.int32)).target_argmax
            assert np.array_equal(got[b, :n], ref), f"call {call}, sequence {b}: differs from the oracle"


def test_static_argmax_rejects_sizes_beyond_its_array():
    import torch
    from paper_2601_12212_b200 import binding
    lib = binding.load()
    x = torch.zeros(16, device="cuda")
    n = torch.ones(16, dtype=torch.int32, device="cuda")
    o = torch.zeros(16, dtype=torch.int32, device="cuda")
    vp = ctypes.c_void_p
    # 9 sequences x 128 nodes = 1152 rows > RESPS_STATIC_MAX_ROWS
    rc = lib.resps_target_argmax_static(vp(n.data_ptr()), 9, 128, 16, vp(x.data_ptr()), 0, 16, vp(o.data_ptr()), None)
    assert rc == binding.RESPS_ERR_CAPACITY and "capacity" in binding.strerror(rc)
    rc = lib.resps_target_argmax_static(vp(n.data_ptr()), 1, 129, 16, vp(x.data_ptr()), 0, 16, vp(o.data_ptr()), None)
    assert rc == binding.RESPS_ERR_UNSUPPORTED_SHAPE
    rc = lib.resps_target_argmax_static(None, 1, 1, 16, vp(x.data_ptr()), 0, 16, vp(o.data_ptr()), None)
    assert rc == binding.RESPS_ERR_INVALID_ARG
