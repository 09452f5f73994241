"""Pins for the oracle's controller step (Algorithm 1: action caching with interval N; Eq. 3 and
Eq. 5: reward = tokens per second, averaged over the interval; Appendix A: the [128, 128] policy)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_12212_b200 import synth


def _weights(rng, F, H, A):
    return (rng.normal(size=(H, F)) / np.sqrt(F), rng.normal(size=H) * 0.1, rng.normal(size=(H, H)) / np.sqrt(H),
            rng.normal(size=H) * 0.1, rng.normal(size=(A, H)) / np.sqrt(H), rng.normal(size=A) * 0.1)


def test_policy_network_equals_the_library_mlp():
    rng = np.random.default_rng(0)
    F, H, A = 96, 128, 17
    w = _weights(rng, F, H, A)
    s = rng.normal(size=F)
    net = torch.nn.Sequential(torch.nn.Linear(F, H), torch.nn.Tanh(), torch.nn.Linear(H, H), torch.nn.Tanh(),
                              torch.nn.Linear(H, A)).double()
    with torch.no_grad():
        for layer, (wi, bi) in zip((net[0], net[2], net[4]), ((w[0], w[1]), (w[2], w[3]), (w[4], w[5]))):
            layer.weight.copy_(torch.from_numpy(wi))
            layer.bias.copy_(torch.from_numpy(bi))
        want = net(torch.from_numpy(s)).numpy()
    np.testing.assert_allclose(oracle.policy_logits(s, *w), want, atol=1e-12)
    # closed form: zero weights leave the output bias
    z = [np.zeros_like(x) for x in w]
    z[5] = w[5]
    np.testing.assert_array_equal(oracle.policy_logits(s, *z), w[5])


def test_action_persistence_and_averaged_reward():
    """The policy is asked at steps 0, N, 2N, ...; in between the cached action is used; the reward
    reported when an interval closes is the mean of (accepted + 1) / seconds over its N steps."""
    rng = np.random.default_rng(1)
    F, H = 24, 128
    actions = np.array(synth.action_space(filtered=True), np.int32)
    w = _weights(rng, F, H, len(actions))
    N = 4
    st = oracle.ControllerState()
    asked, chosen, rewards, per_step = [], [], [], []
    prev = (None, None)
    for step in range(13):
        s = rng.normal(size=F)
        st, act, r_avg, logits, _ = oracle.controller_step(st, s, w, actions, N, 0.0, 0.5, *prev)
        asked.append(logits is not None)
        chosen.append(act)
        if logits is not None:
            assert act == tuple(actions[int(np.argmax(logits))])          # temperature 0: the arg-max action
        if r_avg is not None:
            rewards.append((step, r_avg))
        a, secs = int(rng.integers(0, 6)), float(rng.uniform(1e-3, 2e-3))
        per_step.append((a + 1) / secs)
        prev = (a, secs)
    assert asked == [i % N == 0 for i in range(13)]
    for i in range(13):
        assert chosen[i] == chosen[i - i % N]                            # held for N steps
    assert [s for s, _ in rewards] == [4, 8, 12]
    for s, r in rewards:
        assert r == pytest.approx(np.mean(per_step[s - N:s]), rel=1e-12)
    # every action of the filtered grid respects TT <= k^(d-1) (Appendix A)
    assert all(int(tt) <= int(k) ** (int(d) - 1) for tt, d, k in actions)


def test_sampling_at_temperature_follows_the_softmax():
    rng = np.random.default_rng(2)
    F, H, A = 12, 128, 5
    actions = np.array([(32, 3, 8), (48, 4, 8), (64, 5, 12), (80, 6, 16), (96, 7, 20)], np.int32)
    w = _weights(rng, F, H, A)
    s = rng.normal(size=F)
    T = 1.5
    z = oracle.policy_logits(s, *w) / T
    p = np.exp(z - z.max())
    p /= p.sum()
    counts = np.zeros(A)
    trials = 20000
    for _ in range(trials):
        st, act, _, _, _ = oracle.controller_step(oracle.ControllerState(), s, w, actions, 10, T, rng.uniform(), None, None)
        counts[st.action] += 1
    chi2 = float(((counts - trials * p) ** 2 / (trials * p)).sum())
    assert chi2 < 23.5                                                    # 4 degrees of freedom, p = 1e-4
