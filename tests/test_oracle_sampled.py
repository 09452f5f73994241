"""Pins for the oracle's acceptance under sampling (Section 3.2, "Acceptance Criterion": accept a
draft token with probability min(1, P_T / P_d); Section 4.1, "Lossless Output Fidelity": the output
keeps the target model's distribution)."""
import numpy as np
import pytest

import oracle


def _chain_case(p, q, x, rng, T=1.0):
    """Root plus one drafted token x; the target's distribution after the root is p, the draft's q."""
    V = len(p)
    tl = np.zeros((2, V), np.float32)
    tl[0] = np.log(p) * T
    tl[1] = np.log(np.roll(p, 1)) * T            # after the drafted token (only used when it is accepted)
    dr = (np.log(q) * T).astype(np.float32)[None]
    ua = rng.uniform(size=(4, 2))
    us = rng.uniform(size=4)
    return oracle.verify_accept_sampled(tl, dr, np.array([0, -1], np.int32), np.array([7, x], np.int32),
                                        np.array([-1, 0], np.int32), T, ua, us, path_cap=4)


@pytest.mark.parametrize("T", [1.0, 0.7])
def test_chain_of_sampled_draft_tokens_keeps_the_target_distribution(T):
    """The paper's claim, for the case it states (a chain whose tokens are sampled from the draft
    distribution): the first emitted token is distributed as P_T, whatever P_d is; the acceptance
    rate is sum_v min(P_T(v), P_d(v)).  Chi-square against the exact P_T over 60 000 trials."""
    rng = np.random.default_rng(5)
    V, trials = 6, 60000
    p = rng.dirichlet(np.ones(V) * 0.8)
    q = rng.dirichlet(np.ones(V) * 0.8)
    # float32 logits carry p and q only to 1e-7: take the distributions the oracle really sees
    p = np.exp(np.log(p).astype(np.float32).astype(np.float64)); p /= p.sum()
    q = np.exp(np.log(q).astype(np.float32).astype(np.float64)); q /= q.sum()
    counts = np.zeros(V)
    accepted = 0
    for _ in range(trials):
        x = int(rng.choice(V, p=q))
        r = _chain_case(p, q, x, rng, T)
        first = x if r.accept_len >= 1 else int(r.out_tokens[0])
        assert r.out_tokens[0] == first
        counts[first] += 1
        accepted += r.accept_len >= 1
    chi2 = float(((counts - trials * p) ** 2 / (trials * p)).sum())
    assert chi2 < 25.7, chi2                      # chi-square, 5 degrees of freedom, p = 1e-4
    rate = np.minimum(p, q).sum()
    assert abs(accepted / trials - rate) < 4 * np.sqrt(rate * (1 - rate) / trials)


def test_a_leaf_draws_by_inverse_cdf_in_token_order():
    """No children: the token is drawn from P_T by inverse CDF; against numpy's cumsum + searchsorted."""
    rng = np.random.default_rng(1)
    V = 50
    x = rng.normal(size=V).astype(np.float32) * 2
    p = np.exp(x.astype(np.float64) / 0.9)
    cdf = np.cumsum(p / p.sum())
    for _ in range(300):
        u = rng.uniform()
        r = oracle.verify_accept_sampled(x[None], np.zeros((1, V), np.float32), np.array([-1], np.int32),
                                         np.array([3], np.int32), np.array([-1], np.int32), 0.9,
                                         np.zeros((2, 1)), np.array([u, 0.5]), path_cap=2)
        want = int(np.searchsorted(cdf, u, side="right"))
        assert r.accept_len == 0 and (r.out_tokens[0] == want or r.min_margin < 1e-12)
        assert 0.0 <= r.min_margin <= 1.0


def test_temperature_to_zero_is_the_greedy_walk():
    """As T -> 0 both distributions become one-hot and the rule degenerates to "accept iff the token is
    the target's arg-max": path and tokens equal the greedy oracle's on random trees."""
    rng = np.random.default_rng(9)
    for trial in range(60):
        V, k, d = 40, int(rng.integers(1, 4)), int(rng.integers(1, 5))
        TT = int(rng.integers(2, 14))
        logits = rng.normal(size=(d, k, V)).astype(np.float32) * 3
        t = oracle.tree_expand(5, logits, TT, d, k, 0)
        n = t.n_nodes
        tl = rng.normal(size=(n, V)).astype(np.float32) * 3
        for i in range(n):                                    # make the target agree with a child half of the time
            kids = np.nonzero(t.parent == i)[0]
            if kids.size and rng.uniform() < 0.6:
                tl[i, t.tokens[kids[int(rng.integers(kids.size))]]] = tl[i].max() + 1.0
            tl[i, int(np.argmax(tl[i]))] += 1.0               # a clear winner in every row (at least e^-50 ahead)
        g = oracle.verify_accept(tl, t.tokens, t.parent, path_cap=d + 1)
        # (T = 0.02 on logits of spread 3: neighbouring probabilities are e^-25 apart, nothing underflows)
        s = oracle.verify_accept_sampled(tl, logits.reshape(d * k, V), t.node_rows(d, k, k), t.tokens, t.parent, 0.02,
                                         rng.uniform(0.05, 0.95, size=(d + 1, k)), rng.uniform(0.05, 0.95, size=d + 1),
                                         path_cap=d + 1)
        assert s.accept_len == g.accept_len
        assert np.array_equal(s.path, g.path) and np.array_equal(s.out_tokens, g.out_tokens)


def test_the_decision_flips_exactly_at_alpha_and_the_margin_says_how_close_it_was():
    p = np.array([0.5, 0.3, 0.2])
    q = np.array([0.2, 0.2, 0.6])
    p32 = np.exp(np.log(p).astype(np.float32).astype(np.float64)); p32 /= p32.sum()
    q32 = np.exp(np.log(q).astype(np.float32).astype(np.float64)); q32 /= q32.sum()
    alpha = p32[2] / q32[2]                                   # token 2: P_T / P_d = 1/3
    tl = np.log(np.stack([p, p])).astype(np.float32)
    dr = np.log(q).astype(np.float32)[None]
    args = (tl, dr, np.array([0, -1], np.int32), np.array([9, 2], np.int32), np.array([-1, 0], np.int32), 1.0)
    for delta, accepted in ((-1e-6, True), (1e-6, False)):
        ua = np.full((3, 1), 0.5)
        ua[0, 0] = alpha + delta
        r = oracle.verify_accept_sampled(*args, ua, np.array([0.999, 0.4, 0.4]), path_cap=3)
        assert (r.accept_len == 1) == accepted
        assert r.min_margin == pytest.approx(1e-6, rel=1e-3)
    # rejected: the token comes from the residual max(0, p - q) = (0.3, 0.1, 0) / 0.4, never token 2
    ua = np.full((3, 1), 0.9)
    for u, want in ((0.1, 0), (0.74, 0), (0.76, 1), (0.999, 1)):
        r = oracle.verify_accept_sampled(*args, ua, np.array([u, 0.4, 0.4]), path_cap=3)
        assert r.accept_len == 0 and r.out_tokens[0] == want
