"""Pins for the oracle's routing and permutation (CPU only)."""
import itertools

import numpy as np
import pytest
import torch

from oracle import ftmoe_oracle as O


def _dominates(z, s, u):
    return z[s] > z[u] or (z[s] == z[u] and s < u)


@pytest.mark.parametrize("E,k", [(4, 1), (5, 2), (6, 3), (6, 6)])
def test_topk_is_max_sum_subset(E, k):
    rng = np.random.default_rng(E * 10 + k)
    z = rng.standard_normal((20, E)).astype(np.float32)
    ids, w = O.route(z, k)
    for t in range(z.shape[0]):
        best = max(itertools.combinations(range(E), k), key=lambda c: sum(float(z[t, e]) for e in c))
        assert set(best) == set(int(v) for v in ids[t])


def test_topk_total_order_with_ties_and_signed_zero():
    z = np.array([[1.0, 2.0, 2.0, -0.0, 0.0, 2.0],
                  [0.0, -0.0, 0.0, -0.0, -1.0, -1.0],
                  [3.0, 3.0, 3.0, 3.0, 3.0, 3.0]], dtype=np.float32)
    ids, w = O.route(z, 4)
    assert ids[0].tolist() == [1, 2, 5, 0]
    assert ids[1].tolist() == [0, 1, 2, 3]
    assert ids[2].tolist() == [0, 1, 2, 3]
    np.testing.assert_allclose(w[2], 0.25, atol=1e-7)
    # every selected expert precedes every unselected one in the total order; ids are in that order
    rng = np.random.default_rng(1)
    z = rng.integers(-2, 3, size=(50, 8)).astype(np.float32)   # many ties
    ids, _ = O.route(z, 3)
    for t in range(50):
        sel = [int(v) for v in ids[t]]
        for a, b in zip(sel, sel[1:]):
            assert _dominates(z[t], a, b)
        for u in set(range(8)) - set(sel):
            assert all(_dominates(z[t], s, u) for s in sel)


def test_gate_weights_properties():
    rng = np.random.default_rng(2)
    z = (rng.standard_normal((64, 16)) * 3).astype(np.float32)
    ids, w = O.route(z, 4)
    np.testing.assert_allclose(w.sum(axis=1), 1.0, atol=1e-6)
    assert np.all(w[:, :-1] >= w[:, 1:])
    # k = E is the library softmax
    ids_all, w_all = O.route(z, 16)
    ref = torch.softmax(torch.from_numpy(z).double(), dim=1).numpy()
    np.testing.assert_allclose(w_all, np.take_along_axis(ref, ids_all.astype(np.int64), axis=1), atol=1e-7)
    # "softmax over all experts, renormalised over the selected ones" is the same thing
    two_stage = np.take_along_axis(ref, ids.astype(np.int64), axis=1)
    two_stage = two_stage / two_stage.sum(axis=1, keepdims=True)
    np.testing.assert_allclose(w, two_stage, atol=1e-6)
    # k = 1
    _, w1 = O.route(z, 1)
    assert np.all(w1 == 1.0)
    # shift invariance: power-of-two shifts keep fp32 differences exact for these magnitudes
    ids_s, w_s = O.route((z.astype(np.float64) + 4.0).astype(np.float32), 4)
    assert np.array_equal(ids_s, ids)
    np.testing.assert_allclose(w_s, w, atol=2e-6)
    # permuting the expert columns permutes the ids
    pi = rng.permutation(16)
    ids_p, w_p = O.route(z[:, pi], 4)
    assert np.array_equal(pi[ids_p], ids)
    np.testing.assert_array_equal(w_p, w)


def test_route_rejects_nonfinite():
    z = np.zeros((2, 4), dtype=np.float32)
    z[1, 2] = np.nan
    with pytest.raises(ValueError):
        O.route(z, 2)
    z[1, 2] = np.inf
    with pytest.raises(ValueError):
        O.route(z, 2)


@pytest.mark.parametrize("T,k,E", [(1, 1, 4), (8, 2, 8), (37, 4, 16), (0, 2, 8)])
def test_permute_is_library_stable_sort(T, k, E):
    rng = np.random.default_rng(T + k)
    ids = rng.integers(0, E, size=(T, k)).astype(np.int32)
    count, offset, perm, inv = O.permute(ids, E)
    keys = ids.reshape(-1)
    ref = np.argsort(keys, kind="stable").astype(np.int32)
    assert np.array_equal(perm, ref)
    assert np.array_equal(count, np.bincount(keys, minlength=E))
    assert offset[0] == 0 and np.array_equal(offset[1:], np.cumsum(count))
    assert np.array_equal(inv[perm], np.arange(T * k))
    assert np.array_equal(perm[inv], np.arange(T * k))
    assert np.all(np.diff(keys[perm]) >= 0)
