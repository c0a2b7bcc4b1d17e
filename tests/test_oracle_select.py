"""Pins for the oracle's selective-speculation support (Section 5.1): draft confidence and the
keep-top-(1-alpha) selection.  CPU only; checked against scipy's softmax, closed forms, numpy's
lexsort and the invariants that define such a selection."""
import math

import numpy as np
import pytest
import scipy.special
import torch

import oracle


def _batch(rng, ks, V, dtype=torch.float32):
    qi = np.concatenate([[0], np.cumsum(np.array(ks) + 1)]).astype(np.int32)
    TD = int(sum(ks))
    dl = torch.from_numpy((rng.standard_normal((TD, V)) * 2).astype(np.float32)).to(dtype)
    ids = torch.from_numpy(rng.integers(0, V, size=TD).astype(np.int32))
    return dl, ids, torch.from_numpy(qi)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_confidence_against_scipy_softmax(dtype):
    rng = np.random.default_rng(3)
    ks = [3, 0, 1, 5, 2]
    dl, ids, qi = _batch(rng, ks, 300, dtype)
    cmax, ctok, creq = oracle.draft_confidence(dl, ids, qi)
    q = scipy.special.softmax(dl.double().numpy(), axis=1)
    assert np.allclose(cmax.numpy(), q.max(axis=1), rtol=1e-12)
    assert np.allclose(ctok.numpy(), q[np.arange(len(ids)), ids.numpy()], rtol=1e-12)
    d = 0
    for r, k in enumerate(ks):
        assert math.isclose(float(creq[r]), float(np.prod(q[d:d + k].max(axis=1))), rel_tol=1e-12)
        d += k
    assert float(creq[1]) == 1.0                                  # no drafts: empty product


def test_confidence_closed_forms():
    V = 64
    qi = torch.tensor([0, 3], dtype=torch.int32)
    w = np.arange(1, V + 1, dtype=np.float64)
    rows = np.stack([np.zeros(V), np.log(w)]).astype(np.float32)
    cmax, ctok, creq = oracle.draft_confidence(torch.from_numpy(rows), torch.tensor([5, 9], dtype=torch.int32), qi)
    assert math.isclose(float(cmax[0]), 1.0 / V, rel_tol=1e-12)   # uniform row
    assert math.isclose(float(cmax[1]), V / w.sum(), rel_tol=1e-6)  # logits ln(w): top-1 = w_max / sum w
    assert math.isclose(float(ctok[1]), 10.0 / w.sum(), rel_tol=1e-6)
    assert math.isclose(float(creq[0]), float(cmax[0] * cmax[1]), rel_tol=1e-12)
    # an invalid id is reported and isolated
    cmax2, ctok2, _ = oracle.draft_confidence(torch.from_numpy(rows), torch.tensor([5, V], dtype=torch.int32), qi)
    assert torch.equal(cmax2, cmax) and math.isnan(float(ctok2[1])) and float(ctok2[0]) == float(ctok[0])


def _lexsort_reference(conf, k_in, alpha):
    part = np.nonzero(k_in > 0)[0]
    n_drop = int(math.floor(alpha * len(part)))
    # ascending confidence; among equals the higher index first
    order = part[np.lexsort((-part, conf[part]))]
    k_out = k_in.copy()
    k_out[order[:n_drop]] = 0
    return k_out, n_drop


@pytest.mark.parametrize("alpha", [0.0, 0.15, 0.3, 0.5, 1.0])
def test_selection_against_numpy_lexsort(alpha):
    rng = np.random.default_rng(int(alpha * 100) + 1)
    for B in (1, 7, 64, 257):
        conf = rng.random(B).astype(np.float32)
        conf[rng.integers(0, B, size=B // 3)] = 0.5               # many ties
        k_in = rng.integers(0, 4, size=B).astype(np.int32)
        k_out, n_drop = oracle.select_speculation(torch.from_numpy(conf), torch.from_numpy(k_in), alpha)
        ref, ref_drop = _lexsort_reference(conf, k_in, alpha)
        assert n_drop == ref_drop and np.array_equal(k_out.numpy(), ref)


def test_selection_invariants_and_special_values():
    rng = np.random.default_rng(9)
    B = 200
    conf = rng.random(B).astype(np.float32)
    k_in = np.where(rng.random(B) < 0.8, 3, 0).astype(np.int32)
    N = int((k_in > 0).sum())
    k_out, n_drop = oracle.select_speculation(torch.from_numpy(conf), torch.from_numpy(k_in), 0.3)
    k_out = k_out.numpy()
    assert n_drop == math.floor(0.3 * N)
    dropped = (k_in > 0) & (k_out == 0)
    kept = k_out > 0
    assert dropped.sum() == n_drop and (k_out[kept] == k_in[kept]).all() and (k_out[k_in == 0] == 0).all()
    assert conf[dropped].max() <= conf[kept].min()                # separation
    # ties: the higher index goes first
    conf2 = np.full(6, 0.25, dtype=np.float32)
    k2, nd2 = oracle.select_speculation(torch.from_numpy(conf2), torch.full((6,), 2, dtype=torch.int32), 0.5)
    assert nd2 == 3 and k2.tolist() == [2, 2, 2, 0, 0, 0]
    # the order is total: -0 < +0, +inf above every finite value, a NaN of positive sign above +inf
    conf3 = torch.tensor([0.0, -0.0, float("inf"), float("nan"), 1.0])
    k3, _ = oracle.select_speculation(conf3, torch.ones(5, dtype=torch.int32), 0.4)
    assert k3.tolist() == [0, 0, 1, 1, 1]
    with pytest.raises(oracle.OracleError):
        oracle.select_speculation(torch.zeros(3), torch.ones(3, dtype=torch.int32), 1.5)
    with pytest.raises(oracle.OracleError):
        oracle.select_speculation(torch.zeros(3), torch.ones(3, dtype=torch.int32), float("nan"))


def test_selection_raises_the_mean_confidence_of_what_is_kept():
    # the property Section 5.1 relies on: dropping the lowest-confidence fraction leaves a batch
    # whose mean confidence is at least the original mean
    rng = np.random.default_rng(4)
    conf = rng.beta(2, 2, size=500).astype(np.float32)
    k_in = np.ones(500, dtype=np.int32)
    for alpha in (0.15, 0.3):
        k_out, _ = oracle.select_speculation(torch.from_numpy(conf), torch.from_numpy(k_in), alpha)
        assert conf[k_out.numpy() > 0].mean() > conf.mean()
