"""Edge cases of the CUDA path through the C-ABI, each against the CPU oracle: ties, scalar
(unaligned) logits path, extreme k, clamping of (TT, d, k), ragged batches, poisoned cache
slots, in-place compaction hazards, device status bits and host-side errors."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _imports():
    import oracle
    from paper_2601_12212_b200 import binding, synth
    return oracle, binding, synth


class Bufs:
    def __init__(self, B, T, D1, dev="cuda"):
        i32 = dict(dtype=torch.int32, device=dev)
        self.tokens = torch.full((B, T), -7, **i32)
        self.parent = torch.full((B, T), -7, **i32)
        self.depth = torch.full((B, T), -7, **i32)
        self.pos = torch.full((B, T), -7, **i32)
        self.mask = torch.zeros(B, T, 2, dtype=torch.int64, device=dev)
        self.retrieve = torch.full((B, T, D1), -7, **i32)
        self.n_leaves = torch.zeros(B, **i32)
        self.n_nodes = torch.zeros(B, **i32)


def expand_and_compare(logits, params, roots, max_tt=128, max_k=None, max_d=None, vocab=None,
                       expect_status=0, ld_pad=0, offset=0):
    """logits: list (per sequence) of fp32 [d][k][V]; params: list of (TT, d, k, L)."""
    oracle, binding, synth = _imports()
    B = len(params)
    V = vocab or logits[0].shape[2]
    max_k = max_k or max(p[2] for p in params)
    max_d = max_d or max(p[1] for p in params)
    ctx = binding.Context(8, 2, 64, V, max_batch=B, max_tt=max_tt, max_k=max_k, max_depth=max_d)
    ld_row = V + ld_pad
    flat = torch.zeros(offset + B * max_d * max_k * ld_row, dtype=torch.float32, device="cuda")
    view = flat[offset:].view(B, max_d, max_k, ld_row)
    for s, lg in enumerate(logits):
        d, k = min(lg.shape[0], max_d), min(lg.shape[1], max_k)
        view[s, :d, :k, :V].copy_(torch.from_numpy(np.ascontiguousarray(lg[:d, :k])))
    steps = torch.tensor(params, dtype=torch.int32, device="cuda")
    root = torch.tensor(roots, dtype=torch.int32, device="cuda")
    bufs = Bufs(B, max_tt, max_d + 1)
    for rep in range(2):  # twice: the workspace counters must have reset themselves
        binding.resps_tree_expand(ctx, steps, B, view, max_d * max_k * ld_row, max_k * ld_row, ld_row,
                                  max_d, max_k, root, bufs.tokens, bufs.parent, bufs.depth, bufs.pos,
                                  bufs.mask, bufs.retrieve, bufs.n_leaves, bufs.n_nodes)
        assert ctx.status() == expect_status
        for s, (tt, d, k, L) in enumerate(params):
            tt_c, d_c = min(max(tt, 1), max_tt), min(max(d, 1), max_d)
            k_c = min(max(k, 1), min(V, max_k))
            t = oracle.tree_expand(roots[s], logits[s][:d_c, :max(k_c, 1)], tt_c, d_c, k_c, L,
                                   max_tt=max_tt, ret_stride=max_d + 1)
            n = t.n_nodes
            assert int(bufs.n_nodes[s]) == n and int(bufs.n_leaves[s]) == t.n_leaves
            assert np.array_equal(bufs.tokens[s, :n].cpu().numpy(), t.tokens)
            assert np.array_equal(bufs.parent[s, :n].cpu().numpy(), t.parent)
            assert np.array_equal(bufs.depth[s, :n].cpu().numpy(), t.depth)
            assert np.array_equal(bufs.pos[s, :n].cpu().numpy(), t.position_ids)
            assert np.array_equal(bufs.mask[s, :n].cpu().numpy().view(np.uint64), t.mask)
            assert np.array_equal(bufs.retrieve[s, : t.n_leaves].cpu().numpy(), t.retrieve)
            assert (bufs.tokens[s, n:] == -7).all() and (bufs.retrieve[s, t.n_leaves:] == -7).all()
    ctx.close()


def test_ties_everywhere_all_equal_and_quantised_logits():
    rng = np.random.default_rng(0)
    V = 5000
    flat = np.zeros((3, 4, V), np.float32)                       # every logit equal
    quant = np.round(rng.normal(size=(4, 6, V)) * 2).astype(np.float32)  # many equal values
    quant[quant == 0] = -0.0                                     # signed zeros compare equal
    expand_and_compare([flat, quant], [(40, 3, 4, 10), (100, 4, 6, 0)], [1, 2])


def test_scalar_path_odd_vocab_padded_rows_and_misaligned_base():
    rng = np.random.default_rng(1)
    V = 10007
    lg = (rng.normal(size=(3, 5, V)) * 3).astype(np.float32)
    expand_and_compare([lg], [(30, 3, 5, 7)], [3], ld_pad=3, offset=1)
    expand_and_compare([lg[:, :, :10004]], [(30, 3, 5, 7)], [3], ld_pad=4, offset=4)  # vector path, padded


def test_extreme_k_and_depth():
    rng = np.random.default_rng(2)
    V = 40000
    lg = (rng.normal(size=(8, 32, V)) * 2).astype(np.float32)
    expand_and_compare([lg], [(128, 8, 32, 123)], [9])           # the paper's largest action
    expand_and_compare([lg[:, :1]], [(128, 8, 1, 0)], [9])       # chain
    expand_and_compare([lg[:1, :1]], [(128, 1, 32, 0)], [9])     # star
    expand_and_compare([lg[:1, :1]], [(1, 1, 1, 5)], [9])        # root only
    lg16 = (rng.normal(size=(16, 4, 3000)) * 2).astype(np.float32)
    expand_and_compare([lg16], [(128, 16, 4, 0)], [1])           # deepest tree


def test_tiny_vocab_and_k_equals_vocab():
    rng = np.random.default_rng(3)
    lg = rng.normal(size=(3, 8, 8)).astype(np.float32)
    expand_and_compare([lg], [(64, 3, 8, 0)], [0])


def test_adversarial_ascending_row_every_element_enters_the_list():
    V = 20000
    lg = np.tile(np.arange(V, dtype=np.float32) * 0.001, (2, 3, 1))
    lg[1, 1] = lg[1, 1][::-1]
    expand_and_compare([lg], [(20, 2, 3, 0)], [0])


def test_ragged_batch_and_clamping_sets_status():
    oracle, binding, synth = _imports()
    rng = np.random.default_rng(4)
    V = 3000
    lgs = [(rng.normal(size=(6, 9, V)) * 2).astype(np.float32) for _ in range(4)]
    params = [(16, 3, 4, 100), (80, 6, 9, 4000), (48, 5, 4, 5), (60, 4, 12, 77)]
    # the last sequence asks for k=12 with only 9 slots: clamped to 9 and flagged
    expand_and_compare(lgs, params, [5, 6, 7, 8], max_k=9, max_d=6, max_tt=80,
                       expect_status=binding.RESPS_STATUS_STEP_CLAMPED)
    expand_and_compare(lgs[:3], params[:3], [5, 6, 7], max_k=9, max_d=6, max_tt=80)
    # TT beyond the pool: clamps to 1 + n_cand without any flag ("upper limits")
    expand_and_compare(lgs[:1], [(80, 3, 4, 0)], [1], max_tt=80)


# ------------------------------------------------------------------------ attention
def _attention_case(n, Hq, Hkv, D, L, cap, parent=None, poison=False, seed=0, B=1, max_tt=128, v_scale=1.0,
                    debug=()):
    oracle, binding, synth = _imports()
    from harness import check_attention, u16_to_bf16_cuda, bf16_to_f64
    rng = np.random.default_rng(seed)
    ctx = binding.Context(Hq, Hkv, D, 1000, max_batch=B, max_tt=max_tt, max_k=4, max_depth=4)
    for key, value in debug:
        ctx.debug_set(key, value)
    ns = [n] * B if isinstance(n, int) else n
    Ls = [L] * B if isinstance(L, int) else L
    q = synth.to_bf16_bits(rng.normal(size=(B, max_tt, Hq, D)).astype(np.float32).ravel()).reshape(B, max_tt, Hq, D)
    kc = synth.to_bf16_bits(rng.normal(size=(B, Hkv, cap, D)).astype(np.float32).ravel()).reshape(B, Hkv, cap, D)
    vc = synth.to_bf16_bits((rng.normal(size=(B, Hkv, cap, D)) * v_scale).astype(np.float32).ravel()).reshape(B, Hkv, cap, D)
    masks = np.zeros((B, max_tt, 2), np.uint64)
    for s in range(B):
        par = parent if parent is not None else [-1] + [int(rng.integers(max(0, i - 9), i)) for i in range(1, ns[s])]
        for i in range(ns[s]):
            v, c = 0, i
            while c >= 0:
                v |= 1 << c
                c = par[c]
            masks[s, i] = (v & 0xFFFFFFFFFFFFFFFF, v >> 64)
    big = synth.to_bf16_bits(np.array([1e4], np.float32))[0]
    kc_dev, vc_dev = kc.copy(), vc.copy()
    if poison:
        for s in range(B):
            kc_dev[s, :, Ls[s] + ns[s]:] = big           # slots past the tree: never visible
            vc_dev[s, :, Ls[s] + ns[s]:] = big
    steps = torch.tensor([[ns[s], 1, 1, Ls[s]] for s in range(B)], dtype=torch.int32, device="cuda")
    nn = torch.tensor(ns, dtype=torch.int32, device="cuda")
    dq = u16_to_bf16_cuda(q)
    do = torch.full_like(dq, float("nan"))
    dl = torch.zeros(B, max_tt, Hq, dtype=torch.float32, device="cuda")
    dk, dv = u16_to_bf16_cuda(kc_dev), u16_to_bf16_cuda(vc_dev)
    dm = torch.from_numpy(masks.view(np.int64)).cuda()
    scale = 1.0 / np.sqrt(D)
    for rep in range(2):
        do.fill_(float("nan"))
        binding.resps_tree_attention(ctx, steps, nn, B, dq, do, dl, dk, dv, Hkv * cap * D, cap * D, D,
                                     cap, dm, scale)
        assert ctx.status() == 0
        g = bf16_to_f64(do)
        for s in range(B):
            ref = oracle.tree_attention(q[s, :ns[s]], kc[s], vc[s], Ls[s], masks[s, :ns[s]], scale)
            if v_scale == 1.0:
                check_attention(g[s, :ns[s]], ref)
            else:  # the absolute gate is stated for values of order one: scale it with the values
                check_attention(g[s, :ns[s]] / v_scale, ref / v_scale)
            assert np.isnan(g[s, ns[s]:]).all()
    ctx.close()
    return masks


@pytest.mark.parametrize("n,Hq,Hkv,D,L", [
    (1, 4, 1, 64, 0),        # a single token attending to itself only
    (1, 32, 8, 128, 777),    # plain decode
    (128, 8, 8, 128, 3),     # full tree, MHA, almost no prefix: everything is masked tiles
    (128, 64, 8, 128, 130),  # M = 1024 rows per KV head
    (37, 12, 4, 64, 64),     # prefix ends exactly on a tile boundary
    (60, 32, 8, 128, 1000),
    (17, 6, 2, 128, 2049),
])
def test_attention_shapes_and_boundaries(n, Hq, Hkv, D, L):
    _attention_case(n, Hq, Hkv, D, L, cap=L + 128 + 70, poison=True, seed=n)


@pytest.mark.parametrize("n,Hq,Hkv", [(20, 8, 2), (70, 16, 4)])
def test_attention_large_values_survive_the_split_partials(n, Hq, Hkv):
    """V far beyond the fp16 range, on a prefix long enough to be split: the partial results carry a
    per-row scale."""
    _attention_case(n, Hq, Hkv, 128, 5000, cap=5200, seed=11, v_scale=3.0e5)


@pytest.mark.parametrize("rounds", [2, 3, 4])
def test_attention_work_list_of_several_rounds(rounds):
    """Long sequences may be cut into more items than CTAs (a CTA then takes several, one after the
    other); the library's test-only override forces that on a problem small enough for the oracle."""
    _, binding, _ = _imports()
    dbg = ((binding.RESPS_DEBUG_ATTN_ROUNDS, rounds),)
    _attention_case(40, 16, 4, 128, 9000, cap=9300, seed=rounds, debug=dbg)
    _attention_case([9, 70, 33], 8, 8, 128, [5000, 2500, 7777], cap=8192, seed=rounds, B=3, debug=dbg)


@pytest.mark.parametrize("single_units", [0, 100000])
def test_attention_both_groupings_of_the_work_list(single_units):
    """The work list cuts a call into single row tiles (both halves of a CTA on one tile) while it is small and
    into pairs of row tiles otherwise; the test-only override forces each grouping on shapes that take the
    other one by themselves: a short GQA sequence with several row tiles per KV head, a long one, a ragged batch."""
    _, binding, _ = _imports()
    dbg = ((binding.RESPS_DEBUG_ATTN_SINGLE, single_units),)
    _attention_case(60, 32, 8, 128, 700, cap=1024, seed=11, debug=dbg)
    _attention_case(96, 16, 2, 128, 6000, cap=6400, seed=12, debug=dbg)
    _attention_case([16, 80, 47], 8, 2, 128, [300, 4000, 1500], cap=4608, seed=13, B=3, debug=dbg)


def test_attention_chain_mask_is_causal():
    n = 100
    _attention_case(n, 8, 2, 128, 50, cap=300, parent=list(range(-1, n - 1)), poison=True)


def test_attention_non_ancestor_slots_are_invisible():
    """Huge K/V at a sibling's slot must not reach a node that does not descend from it."""
    oracle, binding, synth = _imports()
    from harness import u16_to_bf16_cuda, bf16_to_f64
    rng = np.random.default_rng(5)
    n, Hq, Hkv, D, L, cap, T = 40, 8, 2, 128, 300, 512, 64
    ctx = binding.Context(Hq, Hkv, D, 1000, max_batch=1, max_tt=T, max_k=4, max_depth=4)
    parent = [-1] + [int(rng.integers(max(0, i - 5), i)) for i in range(1, n)]
    masks = np.zeros((1, T, 2), np.uint64)
    for i in range(n):
        v, c = 0, i
        while c >= 0:
            v |= 1 << c
            c = parent[c]
        masks[0, i, 0] = v
    q = synth.to_bf16_bits(rng.normal(size=T * Hq * D).astype(np.float32)).reshape(1, T, Hq, D)
    kc = synth.to_bf16_bits(rng.normal(size=Hkv * cap * D).astype(np.float32)).reshape(1, Hkv, cap, D)
    vc = synth.to_bf16_bits(rng.normal(size=Hkv * cap * D).astype(np.float32)).reshape(1, Hkv, cap, D)
    steps = torch.tensor([[n, 1, 1, L]], dtype=torch.int32, device="cuda")
    nn = torch.tensor([n], dtype=torch.int32, device="cuda")
    dm = torch.from_numpy(masks.view(np.int64)).cuda()

    def run(kc_, vc_):
        do = torch.zeros(1, T, Hq, D, dtype=torch.bfloat16, device="cuda")
        binding.resps_tree_attention(ctx, steps, nn, 1, u16_to_bf16_cuda(q), do, None,
                                     u16_to_bf16_cuda(kc_), u16_to_bf16_cuda(vc_), Hkv * cap * D,
                                     cap * D, D, cap, dm, 0.088)
        return bf16_to_f64(do)[0, :n]

    base = run(kc, vc)
    victim = 7
    big = synth.to_bf16_bits(np.array([1e4], np.float32))[0]
    k2, v2 = kc.copy(), vc.copy()
    k2[0, :, L + victim] = big
    v2[0, :, L + victim] = big
    out = run(k2, v2)
    for i in range(n):
        descends = (int(masks[0, i, 0]) >> victim) & 1
        if descends:
            assert not np.array_equal(out[i], base[i])
        else:
            assert np.array_equal(out[i], base[i])
    ctx.close()


def test_attention_ragged_batch():
    _attention_case([5, 128, 33, 1], 16, 4, 128, [900, 10, 4000, 123], cap=4200, B=4, poison=True)


def test_attention_batch_of_more_than_a_warp_of_sequences():
    """The work list is built by one warp, a lane per sequence, in rounds of 32: 70 sequences of mixed
    sizes go through three rounds and through the flat combine."""
    rng = np.random.default_rng(3)
    B = 70
    ns = [int(x) for x in rng.choice([1, 2, 7, 20, 33], size=B)]
    ns[0], ns[31], ns[32], ns[69] = 20, 33, 7, 1
    Ls = [int(x) for x in rng.integers(0, 700, size=B)]
    _attention_case(ns, 8, 2, 64, Ls, cap=800, B=B, max_tt=40, seed=9)


def test_attention_overflowing_sequence_is_skipped_and_flagged():
    oracle, binding, synth = _imports()
    ctx = binding.Context(4, 1, 64, 100, max_batch=2, max_tt=16, max_k=4, max_depth=4)
    cap, D = 64, 64
    steps = torch.tensor([[8, 1, 1, 60], [8, 1, 1, 10]], dtype=torch.int32, device="cuda")  # 60+8 > 64
    nn = torch.tensor([8, 8], dtype=torch.int32, device="cuda")
    q = torch.randn(2, 16, 4, D, device="cuda").bfloat16()
    o = torch.full_like(q, float("nan"))
    kc = torch.randn(2, 1, cap, D, device="cuda").bfloat16()
    vc = torch.randn(2, 1, cap, D, device="cuda").bfloat16()
    mask = torch.zeros(2, 16, 2, dtype=torch.int64, device="cuda")
    for i in range(8):
        mask[:, i, 0] = (1 << (i + 1)) - 1
    binding.resps_tree_attention(ctx, steps, nn, 2, q, o, None, kc, vc, cap * D, cap * D, D, cap, mask, 0.125)
    assert ctx.status() == binding.RESPS_STATUS_KV_OVERFLOW
    assert torch.isnan(o[0].float()).all()                  # skipped
    assert not torch.isnan(o[1, :8].float()).any()          # the other sequence ran
    # compaction of the same step: the overflowing sequence is left untouched (no slot past the cache
    # is read or written) and flagged again, the other one is moved
    path = torch.tensor([[0, 3, 7, -1, -1], [0, 2, 5, -1, -1]], dtype=torch.int32, device="cuda")
    alen = torch.tensor([2, 2], dtype=torch.int32, device="cuda")
    k0, v0 = kc.clone(), vc.clone()
    binding.resps_kv_compact(ctx, steps, 2, path, alen, binding.layer_pointer_table([kc]),
                             binding.layer_pointer_table([vc]), 1, cap * D, cap * D, D, cap)
    assert ctx.status() == binding.RESPS_STATUS_KV_OVERFLOW
    assert torch.equal(kc[0], k0[0]) and torch.equal(vc[0], v0[0])
    assert torch.equal(kc[1, :, 11], k0[1, :, 12]) and torch.equal(vc[1, :, 12], v0[1, :, 15])
    # a path entry outside the tree, or a negative prefix that is clamped to 0, is refused or handled too
    bad = torch.tensor([[0, 99, -1, -1, -1], [0, -3, -1, -1, -1]], dtype=torch.int32, device="cuda")
    one = torch.tensor([1, 1], dtype=torch.int32, device="cuda")
    low = torch.tensor([[8, 1, 1, 10], [8, 1, 1, 10]], dtype=torch.int32, device="cuda")
    k1, v1 = kc.clone(), vc.clone()
    binding.resps_kv_compact(ctx, low, 2, bad, one, binding.layer_pointer_table([kc]),
                             binding.layer_pointer_table([vc]), 1, cap * D, cap * D, D, cap)
    assert ctx.status() == binding.RESPS_STATUS_KV_OVERFLOW
    assert torch.equal(kc, k1) and torch.equal(vc, v1)
    ctx.close()


# ------------------------------------------------------------------- verify / compact
def test_verify_accept_ties_and_full_depth_path():
    oracle, binding, synth = _imports()
    V, T, Dm = 50021, 32, 8     # odd vocab: scalar path
    ctx = binding.Context(4, 1, 64, V, max_batch=2, max_tt=T, max_k=4, max_depth=Dm)
    rng = np.random.default_rng(6)
    # sequence 0: a chain of depth 8 fully accepted; sequence 1: ties in the logits
    tokens = np.zeros((2, T), np.int32)
    parent = np.full((2, T), -1, np.int32)
    n = [9, 5]
    tokens[0, :9] = rng.integers(0, V, 9)
    parent[0, :9] = np.arange(-1, 8)
    tokens[1, :5] = [4, 10, 20, 30, 40]
    parent[1, :5] = [-1, 0, 0, 1, 1]
    tl = np.zeros((2, T, V), np.float32)
    tl[0, :9] = rng.normal(size=(9, V))
    for i in range(8):
        tl[0, i, tokens[0, i + 1]] = 50.0
    tl[1, :5] = -1.0
    tl[1, 0, [20, 10]] = 3.0        # tie between two children: the lower id (10) wins
    tl[1, 1, [40, 45]] = 3.0        # tie: 40 wins and is child 4
    steps = torch.tensor([[16, 8, 1, 100], [16, 2, 2, 7]], dtype=torch.int32, device="cuda")
    d = lambda a: torch.from_numpy(a).cuda()
    argm = torch.zeros(2, T, dtype=torch.int32, device="cuda")
    path = torch.zeros(2, Dm + 1, dtype=torch.int32, device="cuda")
    alen = torch.zeros(2, dtype=torch.int32, device="cuda")
    out = torch.zeros(2, Dm + 1, dtype=torch.int32, device="cuda")
    nxt = torch.zeros(2, 4, dtype=torch.int32, device="cuda")
    for rep in range(2):
        binding.resps_verify_accept(ctx, steps, d(np.array(n, np.int32)), 2, d(tl), T * V, V, d(tokens),
                                    d(parent), argm, path, alen, out, nxt)
        for s in range(2):
            acc = oracle.verify_accept(tl[s, :n[s]], tokens[s], parent[s], path_cap=Dm + 1)
            a = acc.accept_len
            assert int(alen[s]) == a
            assert np.array_equal(argm[s, :n[s]].cpu().numpy(), acc.target_argmax)
            assert np.array_equal(path[s, :a + 1].cpu().numpy(), acc.path)
            assert np.array_equal(out[s, :a + 1].cpu().numpy(), acc.out_tokens)
        assert int(alen[0]) == 8 and path[1].tolist()[:3] == [0, 1, 4]
        assert nxt.cpu().tolist() == [[16, 8, 1, 109], [16, 2, 2, 10]]
    ctx.close()


def test_compaction_in_place_hazard_and_strided_cache():
    """Destination slots that are sources of earlier path entries (path = [0,2,3,4,...])."""
    oracle, binding, synth = _imports()
    Hkv, D, cap, B, NL, Dm = 3, 128, 96, 2, 3, 16
    ctx = binding.Context(6, Hkv, D, 100, max_batch=B, max_tt=64, max_k=2, max_depth=Dm)
    rng = np.random.default_rng(7)
    pad = 16                                                    # token stride wider than D
    caches = [torch.from_numpy(rng.integers(-30000, 30000, size=(B, Hkv, cap, D + pad), dtype=np.int16))
              .cuda().view(torch.bfloat16) for _ in range(2 * NL)]
    ks, vs = caches[:NL], caches[NL:]
    host = [c.view(torch.int16).cpu().numpy().view(np.uint16).copy() for c in caches]
    paths = np.full((B, Dm + 1), -1, np.int32)
    paths[0, :17] = [0] + list(range(2, 18))                    # every move overlaps the next
    paths[1, :3] = [0, 5, 9]
    alen = np.array([16, 2], np.int32)
    Ls = [10, 60]
    steps = torch.tensor([[64, 16, 2, Ls[0]], [64, 16, 2, Ls[1]]], dtype=torch.int32, device="cuda")
    binding.resps_kv_compact(ctx, steps, B, torch.from_numpy(paths).cuda(), torch.from_numpy(alen).cuda(),
                             binding.layer_pointer_table(ks), binding.layer_pointer_table(vs), NL,
                             Hkv * cap * (D + pad), cap * (D + pad), D + pad, cap)
    for l in range(NL):
        for s in range(B):
            hk = np.ascontiguousarray(host[l][s, :, :, :D])
            hv = np.ascontiguousarray(host[NL + l][s, :, :, :D])
            oracle.kv_compact(hk, hv, Ls[s], paths[s, : alen[s] + 1])
            gk = ks[l].view(torch.int16).cpu().numpy().view(np.uint16)[s]
            gv = vs[l].view(torch.int16).cpu().numpy().view(np.uint16)[s]
            Ln = Ls[s] + alen[s] + 1
            assert np.array_equal(gk[:, :Ln, :D], hk[:, :Ln]) and np.array_equal(gv[:, :Ln, :D], hv[:, :Ln])
            assert np.array_equal(gk[:, :, D:], host[l][s, :, :, D:])          # padding untouched
            assert np.array_equal(gk[:, Ln:, :D], host[l][s, :, Ln:, :D])      # later slots untouched
    ctx.close()


def test_host_side_errors():
    oracle, binding, synth = _imports()
    ctx = binding.Context(8, 2, 64, 1000, max_batch=2, max_tt=32, max_k=4, max_depth=4)
    z = lambda *s, dt=torch.int32: torch.zeros(*s, dtype=dt, device="cuda")
    steps, nn = z(3, 4), z(3)
    q = z(3, 32, 8, 64, dt=torch.bfloat16)
    kc = z(3, 2, 64, 64, dt=torch.bfloat16)
    mask = z(3, 32, 2, dt=torch.int64)
    with pytest.raises(binding.RespsError) as e:      # batch beyond max_batch
        binding.resps_tree_attention(ctx, steps, nn, 3, q, q, None, kc, kc, 2 * 64 * 64, 64 * 64, 64, 64, mask, 1.0)
    assert e.value.code == binding.RESPS_ERR_CAPACITY
    with pytest.raises(binding.RespsError) as e:      # cache smaller than one tree
        binding.resps_tree_attention(ctx, steps, nn, 1, q, q, None, kc, kc, 2 * 16 * 64, 16 * 64, 64, 16, mask, 1.0)
    assert e.value.code == binding.RESPS_ERR_CAPACITY
    with pytest.raises(binding.RespsError) as e:      # token stride not a multiple of 16 bytes
        binding.resps_tree_attention(ctx, steps, nn, 1, q, q, None, kc, kc, 2 * 64 * 68, 64 * 68, 68, 64, mask, 1.0)
    assert e.value.code == binding.RESPS_ERR_INVALID_ARG
    with pytest.raises(binding.RespsError) as e:      # row stride shorter than the vocabulary
        binding.resps_verify_accept(ctx, steps, nn, 1, z(32, 1000, dt=torch.float32), 32 * 1000, 999,
                                    z(32), z(32), z(32), z(5), z(1), z(5))
    assert e.value.code == binding.RESPS_ERR_INVALID_ARG
    assert ctx.workspace_bytes() > 0
    ctx.close()


def test_attention_shards_by_kv_head_without_any_exchange():
    """Attention is independent per KV head: two "ranks", each with a context for its own half of the
    heads and its own slices of Q and of the caches, produce the halves of the full result (checked
    against the oracle on the full problem).  Nothing has to cross between them."""
    oracle, binding, synth = _imports()
    from harness import check_attention, u16_to_bf16_cuda, bf16_to_f64
    rng = np.random.default_rng(21)
    n, Hq, Hkv, D, L, cap, T = 50, 16, 4, 128, 1500, 1700, 64
    q = synth.to_bf16_bits(rng.normal(size=(1, T, Hq, D)).astype(np.float32).ravel()).reshape(1, T, Hq, D)
    kc = synth.to_bf16_bits(rng.normal(size=(1, Hkv, cap, D)).astype(np.float32).ravel()).reshape(1, Hkv, cap, D)
    vc = synth.to_bf16_bits(rng.normal(size=(1, Hkv, cap, D)).astype(np.float32).ravel()).reshape(1, Hkv, cap, D)
    masks = np.zeros((1, T, 2), np.uint64)
    parent = [-1] + [int(rng.integers(max(0, i - 6), i)) for i in range(1, n)]
    for i in range(n):
        v, c = 0, i
        while c >= 0:
            v |= 1 << c
            c = parent[c]
        masks[0, i, 0] = v
    steps = torch.tensor([[n, 1, 1, L]], dtype=torch.int32, device="cuda")
    nn = torch.tensor([n], dtype=torch.int32, device="cuda")
    dm = torch.from_numpy(masks.view(np.int64)).cuda()
    ref = oracle.tree_attention(q[0, :n], kc[0], vc[0], L, masks[0, :n], 1 / np.sqrt(D))
    out = np.zeros((n, Hq, D))
    ranks = 2
    hq, hkv = Hq // ranks, Hkv // ranks
    for rank in range(ranks):
        ctx = binding.Context(hq, hkv, D, 1000, max_batch=1, max_tt=T, max_k=4, max_depth=4)
        dq = u16_to_bf16_cuda(np.ascontiguousarray(q[:, :, rank * hq:(rank + 1) * hq]))
        dk = u16_to_bf16_cuda(np.ascontiguousarray(kc[:, rank * hkv:(rank + 1) * hkv]))
        dv = u16_to_bf16_cuda(np.ascontiguousarray(vc[:, rank * hkv:(rank + 1) * hkv]))
        do = torch.zeros_like(dq)
        binding.resps_tree_attention(ctx, steps, nn, 1, dq, do, None, dk, dv, hkv * cap * D, cap * D, D, cap, dm,
                                     1 / np.sqrt(D))
        assert ctx.status() == 0
        out[:, rank * hq:(rank + 1) * hq] = bf16_to_f64(do)[0, :n]
        ctx.close()
    check_attention(out, ref)
