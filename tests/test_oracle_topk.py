"""Pins for the oracle's vocabulary top-k, argmax and log-sum-exp (Section 3.2, Draft Tree
Expansion: children are ranked by draft confidence c = softmax probability)."""
import math

import numpy as np
import pytest
import scipy.special
import torch

import oracle


def brute_topk(row, k):
    order = sorted(range(len(row)), key=lambda i: (-float(row[i]), i))
    return [order[r] for r in range(k)]


@pytest.mark.parametrize("seed", range(8))
def test_topk_matches_full_sort_with_ties(seed):
    rng = np.random.default_rng(seed)
    V = int(rng.integers(5, 200))
    # few distinct values => many ties; the order among equals is by id
    row = rng.integers(-3, 4, size=V).astype(np.float32)
    for k in (1, 2, min(7, V), V):
        val, idx, _ = oracle.topk_lse(row, k)
        assert idx.tolist() == brute_topk(row, k)
        assert np.array_equal(val, row[idx])


def test_k1_is_argmax_first_occurrence_and_kV_is_sort():
    rng = np.random.default_rng(1)
    row = rng.normal(size=301).astype(np.float32)
    row[17] = row[250] = row.max() + 1  # tie for the maximum
    _, idx, _ = oracle.topk_lse(row, 1)
    assert idx[0] == 17 == int(np.argmax(row))
    _, idx, _ = oracle.topk_lse(row, row.size)
    assert idx.tolist() == brute_topk(row, row.size)


def test_all_equal_row_gives_lowest_ids():
    row = np.full(64, 2.5, np.float32)
    val, idx, lse = oracle.topk_lse(row, 9)
    assert idx.tolist() == list(range(9))
    assert lse == pytest.approx(2.5 + math.log(64), abs=1e-12)


@pytest.mark.parametrize("seed", range(4))
def test_against_library_topk_on_distinct_values(seed):
    rng = np.random.default_rng(100 + seed)
    row = rng.permutation(5000).astype(np.float32) * 0.01 - 7
    k = 32
    val, idx, _ = oracle.topk_lse(row, k)
    tv, ti = torch.topk(torch.from_numpy(row), k)
    assert idx.tolist() == ti.tolist()
    assert np.array_equal(val, tv.numpy())


def test_lse_closed_forms():
    V = 1000
    # uniform row: every log-prob is -log V
    row = np.full(V, -1.25, np.float32)
    val, idx, lse = oracle.topk_lse(row, 3)
    assert val[0] - lse == pytest.approx(-math.log(V), abs=1e-12)
    # one dominant entry: log-prob -> 0 from below
    row = np.zeros(V, np.float32)
    row[123] = 80.0
    val, idx, lse = oracle.topk_lse(row, 1)
    assert idx[0] == 123
    logp = float(val[0]) - lse
    assert logp <= 0.0 and logp == pytest.approx(-(V - 1) * math.exp(-80.0), abs=1e-30)
    # two-point distribution with probabilities 0.25 / 0.75
    row = np.array([math.log(0.25), math.log(0.75)], np.float32)
    val, idx, lse = oracle.topk_lse(row, 2)
    p = np.exp(val.astype(np.float64) - lse)
    assert idx.tolist() == [1, 0]
    assert p[0] / p[1] == pytest.approx(math.exp(float(row[1]) - float(row[0])), rel=1e-12)
    assert p.sum() == pytest.approx(1.0, abs=1e-12)


@pytest.mark.parametrize("seed", range(4))
def test_probabilities_sum_to_one_and_match_library_logsumexp(seed):
    rng = np.random.default_rng(seed)
    row = (rng.normal(size=4096) * 6).astype(np.float32)
    val, idx, lse = oracle.topk_lse(row, row.size)
    assert np.exp(val.astype(np.float64) - lse).sum() == pytest.approx(1.0, abs=1e-12)
    assert lse == pytest.approx(float(scipy.special.logsumexp(row.astype(np.float64))), abs=1e-12)


def test_large_magnitudes_do_not_overflow():
    row = np.array([3.0e4, 3.0e4 - 1, -3.0e4], np.float32)
    _, _, lse = oracle.topk_lse(row, 1)
    assert lse == pytest.approx(3.0e4 + math.log(1 + math.exp(-1.0)), abs=1e-9)
