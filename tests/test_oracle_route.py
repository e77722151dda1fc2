"""Pins for the CPU checker's router / Top-K / permutation (paper Sections 1 and 2.1: a
trained router sends each token to its Top-K experts).  Expected values come from closed
forms, library routines (scipy softmax, numpy stable argsort) and brute force."""
import itertools

import numpy as np
import pytest
from scipy.special import softmax

import oracle


def _rand(T, d, E, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((T, d)).astype(np.float32)
    Wr = (rng.standard_normal((d, E)) * 0.2).astype(np.float32)
    return x, Wr


def test_hand_example():
    # x = e0 picks row 0 of Wr as logits: z = [0, ln2, ln4, ln1] -> softmax = [1,2,4,1]/8
    Wr = np.zeros((3, 4), dtype=np.float32)
    Wr[0] = np.log(np.array([1.0, 2.0, 4.0, 1.0])).astype(np.float32)
    x = np.array([[1.0, 0.0, 0.0]], dtype=np.float32)
    ids, gates, logits = oracle.route(x, Wr, None, 2, renorm=False)
    assert ids.tolist() == [[2, 1]]
    np.testing.assert_allclose(gates, [[0.5, 0.25]], rtol=1e-6)
    ids, gates, _ = oracle.route(x, Wr, None, 2, renorm=True)
    np.testing.assert_allclose(gates, [[2.0 / 3.0, 1.0 / 3.0]], rtol=1e-6)
    # ties go to the lower index: experts 0 and 3 have equal logits
    ids, _, _ = oracle.route(x, Wr, None, 4, renorm=False)
    assert ids.tolist() == [[2, 1, 0, 3]]
    # bias is added to the logits: +ln8 on expert 3 makes it the winner with p = 8/15
    bias = np.array([0, 0, 0, np.log(8.0)], dtype=np.float32)
    ids, gates, _ = oracle.route(x, Wr, bias, 1, renorm=False)
    assert ids.tolist() == [[3]]
    np.testing.assert_allclose(gates, [[8.0 / 15.0]], rtol=1e-6)
    # per-token bias [T][E]
    x2 = np.repeat(x, 2, axis=0)
    bias2 = np.stack([np.zeros(4, dtype=np.float32), bias])
    ids, _, _ = oracle.route(x2, Wr, bias2, 1, renorm=False)
    assert ids.tolist() == [[2], [3]]


@pytest.mark.parametrize("E,k", [(1, 1), (4, 1), (4, 2), (8, 2), (8, 8), (33, 3)])
def test_against_library_softmax_and_argsort(E, k):
    x, Wr = _rand(9, 16, E, E * 10 + k)
    ids, gates, logits = oracle.route(x, Wr, None, k, renorm=False)
    z = (x.astype(np.float64) @ Wr.astype(np.float64)).astype(np.float32)
    assert np.array_equal(logits, z)
    p = softmax(z.astype(np.float64), axis=1)
    order = np.argsort(-z, axis=1, kind="stable")[:, :k]
    assert np.array_equal(ids, order)
    np.testing.assert_allclose(gates, np.take_along_axis(p, order, axis=1), rtol=1e-6)
    ids2, gates2, _ = oracle.route(x, Wr, None, k, renorm=True)
    assert np.array_equal(ids2, ids)
    np.testing.assert_allclose(gates2.sum(axis=1), 1.0, rtol=1e-6)  # renormalised gates sum to one
    sel = np.take_along_axis(p, order, axis=1)
    np.testing.assert_allclose(gates2, sel / sel.sum(axis=1, keepdims=True), rtol=1e-6)
    if E == 1:
        assert np.all(gates == 1.0) and np.all(gates2 == 1.0)
    if k == E:  # selecting everything: renormalised gates are the full softmax
        np.testing.assert_allclose(gates2, np.take_along_axis(p, order, axis=1), rtol=1e-6)


def test_expert_axis_permutation_equivariance():
    x, Wr = _rand(12, 24, 6, 5)
    ids, gates, _ = oracle.route(x, Wr, None, 2, renorm=True)
    for perm in itertools.islice(itertools.permutations(range(6)), 0, 720, 97):
        perm = np.array(perm)
        ids_p, gates_p, _ = oracle.route(x, Wr[:, perm], None, 2, renorm=True)
        assert np.array_equal(perm[ids_p], ids)
        np.testing.assert_allclose(gates_p, gates, rtol=1e-6)


@pytest.mark.parametrize("T,k,E", [(1, 1, 4), (7, 2, 5), (64, 1, 32), (300, 2, 8), (5, 1, 128)])
def test_permutation_properties_and_library_sort(T, k, E):
    rng = np.random.default_rng(T + k + E)
    ids = rng.integers(0, E, size=(T, k)).astype(np.int32)
    counts, off, perm = oracle.permute(ids, E)
    flat = ids.reshape(-1)
    assert np.array_equal(counts, np.bincount(flat, minlength=E))
    assert counts.sum() == T * k
    assert np.array_equal(off, np.concatenate([[0], np.cumsum(counts)]))
    assert np.array_equal(np.sort(perm), np.arange(T * k))           # a bijection
    assert np.all(np.diff(flat[perm]) >= 0)                          # grouped by expert
    for e in range(E):                                               # stable inside an expert
        seg = perm[off[e]:off[e + 1]]
        assert np.all(np.diff(seg) > 0)
    assert np.array_equal(perm, np.argsort(flat, kind="stable"))


def test_permute_rejects_bad_ids():
    with pytest.raises(ValueError):
        oracle.permute(np.array([[0], [4]], dtype=np.int32), 4)
