"""Pins for the oracle's softmax / confidence / top-k (Eq. 2; Section 3.2)."""
import numpy as np
import pytest
from scipy.special import logsumexp, softmax

import oracle


def test_full_sort_on_tiny_vocab_and_probabilities_sum_to_one():
    rng = np.random.default_rng(0)
    V = 37
    l = np.round(rng.standard_normal((50, V)) * 2).astype(np.float32)  # rounding creates ties
    conf, idx, prob, lse = oracle.confidence_topk(l, V)
    for r in range(l.shape[0]):
        order = np.lexsort((np.arange(V), -l[r]))  # logit descending, index ascending
        assert np.array_equal(idx[r], order)
    assert np.abs(prob.sum(1) - 1).max() < 1e-12
    p = softmax(l.astype(np.float64), axis=1)
    assert np.abs(np.take_along_axis(p, idx.astype(np.int64), 1) - prob).max() < 1e-14
    assert np.abs(conf - p.max(1)).max() < 1e-14
    assert np.abs(lse - logsumexp(l.astype(np.float64), axis=1)).max() < 1e-12
    assert np.abs(conf - np.exp(l.max(1).astype(np.float64) - lse)).max() < 1e-13
    assert np.array_equal(conf, prob[:, 0])


def test_all_equal_logits():
    V, k = 100, 5
    conf, idx, prob, lse = oracle.confidence_topk(np.full((2, V), 1.5, np.float32), k)
    assert np.array_equal(idx, np.tile(np.arange(k), (2, 1)))
    assert np.abs(prob - 1.0 / V).max() < 1e-15 and np.abs(conf - 1.0 / V).max() < 1e-15
    assert np.abs(lse - (1.5 + np.log(V))).max() < 1e-13


def test_planted_peak_closed_form():
    V, delta = 1000, 6.0
    l = np.zeros((1, V), np.float32)
    l[0, 123] = delta
    conf, idx, prob, _ = oracle.confidence_topk(l, 3)
    p = np.exp(delta) / (np.exp(delta) + V - 1)
    assert idx[0].tolist() == [123, 0, 1]
    assert abs(conf[0] - p) < 1e-14 and abs(prob[0, 1] - (1 - p) / (V - 1)) < 1e-15


def test_duplicate_maxima_lowest_index_first():
    l = np.zeros((1, 64), np.float32)
    l[0, [40, 7, 21]] = 3.0
    l[0, 5] = 2.0
    _, idx, prob, _ = oracle.confidence_topk(l, 4)
    assert idx[0].tolist() == [7, 21, 40, 5]
    assert prob[0, 0] == prob[0, 1] == prob[0, 2] > prob[0, 3]


def test_minus_inf_logits_are_last_with_zero_probability():
    l = np.array([[1.0, -np.inf, -np.inf, 0.0]], np.float32)
    _, idx, prob, _ = oracle.confidence_topk(l, 4)
    assert idx[0].tolist() == [0, 3, 1, 2] and prob[0, 2] == 0 and prob[0, 3] == 0


def test_vocabulary_permutation():
    rng = np.random.default_rng(3)
    V, k = 500, 4
    l = rng.standard_normal((20, V)).astype(np.float32)  # continuous: no ties
    perm = rng.permutation(V)
    _, i1, p1, _ = oracle.confidence_topk(l, k)
    _, i2, p2, _ = oracle.confidence_topk(l[:, perm], k)
    assert np.array_equal(perm[i2], i1) and np.abs(p1 - p2).max() < 1e-14


def test_bf16_sized_row_against_scipy():
    import torch
    g = torch.Generator().manual_seed(0)
    l = (torch.randn((3, 126464), generator=g) * 3).bfloat16().float().numpy()
    conf, idx, prob, lse = oracle.confidence_topk(l, 3)
    p = softmax(l.astype(np.float64), axis=1)
    for r in range(3):
        order = np.lexsort((np.arange(l.shape[1]), -l[r]))[:3]
        assert np.array_equal(idx[r], order)
        assert np.abs(p[r, order] - prob[r]).max() < 1e-13
