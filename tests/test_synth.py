"""Host-side checks of the seeded input generators and the workload table."""
import numpy as np
import torch

from paper_2601_12212_b200 import synth


def test_action_space_size_and_filter():
    """Appendix A: 6 x 6 x 5 = 180 combinations; the filter keeps TT <= k**(d-1)."""
    full = synth.action_space()
    assert len(full) == 180 and len(set(full)) == 180
    kept = synth.action_space(filtered=True)
    assert all(tt <= k ** (d - 1) for tt, d, k in kept)
    assert set(full) - set(kept) == {(tt, d, k) for tt, d, k in full if tt > k ** (d - 1)}
    assert max(tt for tt, _, _ in full) <= synth.MAX_TT
    assert max(k for _, _, k in full) <= synth.MAX_K and max(d for _, d, _ in full) <= synth.MAX_D


def test_streams_are_deterministic_and_distinct():
    a = synth.uniform(synth.stream_key(0, 1, 2), 1000)
    b = synth.uniform(synth.stream_key(0, 1, 2), 1000)
    c = synth.uniform(synth.stream_key(0, 1, 3), 1000)
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    assert np.array_equal(synth.bits(synth.stream_key(5), 10, offset=7),
                          synth.bits(synth.stream_key(5), 17)[7:])
    assert 0 < a.min() and a.max() < 1 and abs(a.mean() - 0.5) < 0.05
    z = synth.normal(synth.stream_key(9), 200000)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01


def test_bf16_rounding_matches_library_cast():
    x = (np.random.default_rng(0).normal(size=10000) * 3).astype(np.float32)
    ours = synth.to_bf16_bits(x)
    lib = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, lib)
    assert np.array_equal(synth.bf16_bits_to_f32(ours),
                          torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_peaked_rows_have_top1_probability_point_seven():
    w = synth.WORKLOADS[3]
    x = synth.draft_logits(w, step=2, seq=0, d=2, k=3).astype(np.float64)
    p = np.exp(x - x.max(-1, keepdims=True))
    p /= p.sum(-1, keepdims=True)
    np.testing.assert_allclose(p.max(-1), 0.7, atol=1e-5)


def test_target_logits_peak_follows_children():
    w = synth.WORKLOADS[1]
    tokens = np.array([5, 10, 11, 12], np.int32)
    parent = np.array([-1, 0, 0, 1], np.int32)
    agree = synth.target_logits(w, 0, 0, tokens, parent, 4, 1.0).argmax(-1)
    assert agree[0] == 10 and agree[1] == 12          # first child of nodes 0 and 1
    never = synth.target_logits(w, 0, 0, tokens, parent, 4, 0.0).argmax(-1)
    assert never[0] not in (10, 11) and never[1] != 12


def test_schedule_holds_draws_and_stays_in_grid():
    w = synth.WORKLOADS[5]
    seen = set()
    for seq in range(w.batch):
        for step in range(0, 40, 4):
            p = synth.step_params(w, step, seq)
            assert all(synth.step_params(w, step + i, seq) == p for i in range(4))
            assert p[0] in synth.GRID_TT and p[1] in synth.GRID_D and p[2] in synth.GRID_K
            seen.add(p)
        assert 1024 <= synth.initial_prefix(w, seq) <= 8192
        assert 0.5 <= synth.agreement_prob(w, seq) <= 0.9
    assert len(seen) > 20
    assert synth.step_params(synth.WORKLOADS[2], 17, 0) == (60, 7, 10)
