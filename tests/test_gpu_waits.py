"""Every device-side wait of the library is bounded: when it runs out the kernel flags
RESPS_STATUS_WAIT_TIMEOUT, finishes its protocol and returns, and the context serves the next call.
Exercised with the test build of the library (millisecond limits; one copy can be left out so that
a wait for it really runs out) on tiny single-CTA cases.  Nothing here faults or waits without a
limit: the skipped copy is simply never issued, every wait for it gives up after about a
millisecond, and every copy that was issued is waited for before the CTA leaves."""
import ctypes

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

DROP_KEY, DROP_ATTENTION_V, DROP_SCAN_CHUNK = 100, 1, 2


@pytest.fixture(scope="module")
def waitlib():
    """The binding pointed at the test build (its own shared library), restored afterwards."""
    from paper_2601_12212_b200 import binding, build
    path = build.build(wait_test=True)
    saved = (binding._lib, binding.LIB_PATH)
    binding._lib, binding.LIB_PATH = None, path
    binding.load()
    yield binding
    binding._lib, binding.LIB_PATH = saved


def _attention_inputs(binding, synth, n, Hq, Hkv, D, L, cap, T):
    rng = np.random.default_rng(4)
    q = synth.to_bf16_bits(rng.normal(size=(1, T, Hq, D)).astype(np.float32).ravel()).reshape(1, T, Hq, D)
    kc = synth.to_bf16_bits(rng.normal(size=(1, Hkv, cap, D)).astype(np.float32).ravel()).reshape(1, Hkv, cap, D)
    vc = synth.to_bf16_bits(rng.normal(size=(1, Hkv, cap, D)).astype(np.float32).ravel()).reshape(1, Hkv, cap, D)
    masks = np.zeros((1, T, 2), np.uint64)
    for i in range(n):
        masks[0, i, 0] = (1 << (i + 1)) - 1          # a chain
    return q, kc, vc, masks


def test_attention_wait_runs_out_and_the_context_recovers(waitlib):
    import oracle
    from harness import check_attention, u16_to_bf16_cuda, bf16_to_f64
    from paper_2601_12212_b200 import synth
    binding = waitlib
    n, Hq, Hkv, D, L, cap, T = 4, 4, 1, 64, 20, 64, 16       # one work item, one key tile: a single CTA has work
    ctx = binding.Context(Hq, Hkv, D, 100, max_batch=1, max_tt=T, max_k=4, max_depth=4)
    q, kc, vc, masks = _attention_inputs(binding, synth, n, Hq, Hkv, D, L, cap, T)
    steps = torch.tensor([[n, 1, 1, L]], dtype=torch.int32, device="cuda")
    nn = torch.tensor([n], dtype=torch.int32, device="cuda")
    dq, dk, dv = u16_to_bf16_cuda(q), u16_to_bf16_cuda(kc), u16_to_bf16_cuda(vc)
    dm = torch.from_numpy(masks.view(np.int64)).cuda()
    do = torch.zeros_like(dq)

    def call():
        binding.resps_tree_attention(ctx, steps, nn, 1, dq, do, None, dk, dv, Hkv * cap * D, cap * D, D, cap, dm, 0.125)

    ctx.debug_set(DROP_KEY, DROP_ATTENTION_V)     # the V tile is never fetched: whoever waits for it gives up
    call()
    torch.cuda.synchronize()                      # the call returns
    assert ctx.status() & binding.RESPS_STATUS_WAIT_TIMEOUT
    ctx.debug_set(DROP_KEY, 0)
    do.fill_(float("nan"))
    call()                                        # the same context, a complete call
    assert ctx.status() == 0
    ref = oracle.tree_attention(q[0, :n], kc[0], vc[0], L, masks[0, :n], 0.125)
    check_attention(bf16_to_f64(do)[0, :n], ref)
    ctx.close()


def test_scan_wait_runs_out_and_the_context_recovers(waitlib):
    import oracle
    binding = waitlib
    V, k = 3 * 8192, 4
    ctx = binding.Context(4, 1, 64, V, max_batch=1, max_tt=8, max_k=k, max_depth=2)
    ctx.debug_set(binding.RESPS_DEBUG_SCAN_SLICES, 1)       # one CTA walks the row's three chunks
    rng = np.random.default_rng(8)
    logits = rng.normal(size=(1, 1, 1, V)).astype(np.float32)
    i32 = dict(dtype=torch.int32, device="cuda")
    steps = torch.tensor([[5, 1, k, 0]], **i32)
    dl = torch.from_numpy(logits).cuda()
    root = torch.tensor([3], **i32)
    outs = [torch.full((1, 8), -7, **i32) for _ in range(4)]
    mask = torch.zeros(1, 8, 2, dtype=torch.int64, device="cuda")
    ret = torch.full((1, 8, 3), -7, **i32)
    nl, nn = torch.zeros(1, **i32), torch.zeros(1, **i32)

    def call():
        binding.resps_tree_expand(ctx, steps, 1, dl, V, V, V, 1, 1, root, *outs, mask, ret, nl, nn)

    ctx.debug_set(DROP_KEY, DROP_SCAN_CHUNK)      # the second chunk is never fetched
    call()
    torch.cuda.synchronize()
    assert ctx.status() & binding.RESPS_STATUS_WAIT_TIMEOUT
    ctx.debug_set(DROP_KEY, 0)
    call()
    assert ctx.status() == 0
    t = oracle.tree_expand(3, logits[0], 5, 1, k, 0, max_tt=8, ret_stride=3)
    assert int(nn[0]) == t.n_nodes == 5
    assert np.array_equal(outs[0].cpu().numpy()[0, :5], t.tokens)
    assert np.array_equal(outs[1].cpu().numpy()[0, :5], t.parent)
    ctx.close()
