"""Pins for the oracle's top-k / top-p filtering (CPU only): an independent numpy restatement by
argsort and cumulative sums, hand-worked rows, limits that switch the filters off, ties kept
together, the output law of speculative sampling under filtering, and isolation of bad values."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

import oracle


def _numpy_filter(x, tau, top_k, top_p):
    """Value-threshold top-k then top-p, written with argsort / cumsum / unique."""
    x = x.astype(np.float64)
    V = len(x)
    keep = np.ones(V, dtype=bool)
    if 1 <= top_k < V:
        keep = x >= np.sort(x)[::-1][top_k - 1]
    if top_p < 1.0:
        e = np.where(keep, np.exp((x - x.max()) / tau), 0.0)
        vals = np.unique(x[keep])[::-1]                       # distinct kept values, descending
        group_mass = np.array([e[x == v].sum() for v in vals])
        cum = np.cumsum(group_mass)
        idx = int(np.argmax(cum >= top_p * group_mass.sum()))
        keep &= x >= vals[idx]
    e = np.where(keep, np.exp((x - x.max()) / tau), 0.0)
    return e / e.sum(), int(keep.sum())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_filtered_row_against_numpy(dtype):
    rng = np.random.default_rng(17)
    for trial in range(60):
        V = int(rng.integers(5, 400))
        row = torch.from_numpy((rng.standard_normal(V) * 2).astype(np.float32)).to(dtype)   # bf16 rows carry ties
        tau = float(rng.choice([0.5, 1.0, 1.7]))
        top_k = int(rng.choice([0, 1, 3, V // 2, V, V + 5]))
        top_p = float(rng.choice([1.0, 0.95, 0.5, 0.1]))
        p, kept, margin = oracle.filtered_row(row, tau, top_k, top_p)
        if margin < 1e-9:
            continue                                              # a crossing this close is decided by rounding order
        ref, ref_kept = _numpy_filter(row.float().numpy(), tau, top_k, top_p)
        assert kept == ref_kept and np.allclose(p.numpy(), ref, rtol=1e-12, atol=0), (trial, V, top_k, top_p)


def test_hand_worked_rows():
    w = np.array([0.05, 0.5, 0.15, 0.3])
    row = torch.tensor(np.log(w), dtype=torch.float32)
    p, kept, margin = oracle.filtered_row(row, 1.0, 0, 0.8)          # 0.5 + 0.3 = 0.8 reaches 0.8 ... in binary it may not
    assert kept in (2, 3)
    p, kept, margin = oracle.filtered_row(row, 1.0, 0, 0.79)
    assert kept == 2 and np.allclose(p.numpy(), [0, 0.625, 0, 0.375], atol=1e-7) and margin == pytest.approx(0.01, abs=1e-6)
    p, kept, _ = oracle.filtered_row(row, 1.0, 0, 0.81)
    assert kept == 3 and np.allclose(p.numpy(), [0, 0.5 / 0.95, 0.15 / 0.95, 0.3 / 0.95], atol=1e-7)
    p, kept, _ = oracle.filtered_row(row, 1.0, 2, 1.0)
    assert kept == 2 and np.allclose(p.numpy(), [0, 0.625, 0, 0.375], atol=1e-7)
    # top-k first, then top-p on the survivors: of {0.5, 0.3, 0.15} renormalised, 0.5/0.95 = 0.526 < 0.6 <= 0.842
    p, kept, _ = oracle.filtered_row(row, 1.0, 3, 0.6)
    assert kept == 2
    # temperature acts before the nucleus: at tau = 2 the law is flatter and 0.79 needs three tokens
    s = np.sqrt(w) / np.sqrt(w).sum()
    assert np.sort(s)[::-1][:2].sum() < 0.79
    assert oracle.filtered_row(row, 2.0, 0, 0.79)[1] == 3


def test_limits_and_ties():
    g = torch.Generator().manual_seed(0)
    row = torch.randn(300, generator=g)
    base = oracle.softmax_row(row, tau=0.8)
    for top_k, top_p in ((0, 1.0), (300, 1.0), (-3, 1.0), (10 ** 6, 1.0)):
        p, kept, margin = oracle.filtered_row(row, 0.8, top_k, top_p)
        assert kept == 300 and torch.equal(p, base) and math.isinf(margin)
    am = int(torch.argmax(row))
    for top_k, top_p in ((1, 1.0), (0, 1e-9)):
        p, kept, _ = oracle.filtered_row(row, 0.8, top_k, top_p)
        assert kept == 1 and float(p[am]) == 1.0
    # ties at the k-th value are all kept; a nucleus ending inside a tie keeps the whole tie
    tied = torch.tensor([1.0, 3.0, 2.0, 2.0, 2.0, 0.0])
    p, kept, _ = oracle.filtered_row(tied, 1.0, 2, 1.0)
    assert kept == 4 and float(p[0]) == 0.0 and float(p[2]) == float(p[3]) == float(p[4])
    p, kept, _ = oracle.filtered_row(tied, 1.0, 0, 0.6)
    assert kept == 4


def _requests(T, Dr, n_trials, tau, top_k, top_p, seed):
    rng = np.random.default_rng(seed)
    k, V = Dr.shape
    q = np.stack([_numpy_filter(Dr[i], tau, top_k, top_p)[0] for i in range(k)])
    ids = np.stack([rng.choice(V, size=n_trials, p=q[i]) for i in range(k)], axis=1)
    uni = lambda n: torch.from_numpy(rng.integers(0, 1 << 24, size=n).astype(np.float32) / float(1 << 24))
    qi = torch.arange(0, (n_trials + 1) * (k + 1), k + 1, dtype=torch.int32)
    return (torch.from_numpy(np.tile(T, (n_trials, 1))), torch.from_numpy(np.tile(Dr, (n_trials, 1))),
            torch.from_numpy(ids.reshape(-1).astype(np.int32)), qi, uni(n_trials * k), uni(n_trials))


@pytest.mark.parametrize("top_k,top_p", [(5, 1.0), (0, 0.7), (8, 0.8)])
def test_output_law_is_the_filtered_target_law(top_k, top_p):
    V, k, n_trials, tau = 16, 2, 200_000, 0.9
    rng = np.random.default_rng(top_k + 3)
    T = (rng.standard_normal((k + 1, V)) * 0.8).astype(np.float32)
    Dr = (T[:k] + rng.standard_normal((k, V)) * 0.5).astype(np.float32)
    assert all(2 <= _numpy_filter(T[i], tau, top_k, top_p)[1] < V for i in range(k + 1))      # the filter bites, and leaves a law to test
    tl, dl, ids, qi, ua, us = _requests(T, Dr, n_trials, tau, top_k, top_p, seed=5)
    res = oracle.rejection_sample(tl, dl, ids, qi, ua, us, temperature=torch.full((n_trials,), tau),
                                  top_k=torch.full((n_trials,), top_k, dtype=torch.int32), top_p=torch.full((n_trials,), top_p))
    toks = res.out_tokens.view(n_trials, k + 1).numpy()
    for pos in (0, 1):
        target = _numpy_filter(T[pos], tau, top_k, top_p)[0]
        sel = res.accepted_len.numpy() >= pos
        hist = np.bincount(toks[sel, pos], minlength=V)
        assert hist[target == 0].sum() == 0                       # nothing outside the kept set is ever emitted
        nz = target > 0
        assert scipy.stats.chisquare(hist[nz], target[nz] * sel.sum()).pvalue > 1e-3
    # the unfiltered target law is rejected at this sample size
    full = scipy.special.softmax(T[0].astype(np.float64) / tau)
    assert scipy.stats.chisquare(np.bincount(toks[:, 0], minlength=V) + 1e-9, full * n_trials).pvalue < 1e-6


def test_draft_outside_the_target_set_is_rejected_and_bad_values_isolated():
    V = 10
    T = torch.tensor([[5.0, 4.0, 0, 0, 0, 0, 0, 0, 0, 0]] * 2)
    Dr = torch.tensor([[0.0, 0, 0, 0, 0, 0, 0, 0, 9.0, 0]])
    qi = torch.tensor([0, 2], dtype=torch.int32)
    res = oracle.rejection_sample(T, Dr, torch.tensor([8], dtype=torch.int32), qi, torch.tensor([0.0]), torch.tensor([0.0]),
                                  top_k=torch.tensor([2], dtype=torch.int32))
    assert int(res.accepted_len[0]) == 0 and float(res.rho[0]) == 0.0 and int(res.out_tokens[0]) in (0, 1)
    # invalid nucleus masses are per-request errors
    rng = np.random.default_rng(1)
    B, k = 5, 2
    tl = torch.from_numpy(rng.standard_normal((B * 3, V)).astype(np.float32))
    dl = torch.from_numpy(rng.standard_normal((B * 2, V)).astype(np.float32))
    ids = torch.from_numpy(rng.integers(0, V, size=B * 2).astype(np.int32))
    qi = torch.arange(0, (B + 1) * 3, 3, dtype=torch.int32)
    ua, us = torch.rand(B * 2), torch.rand(B)
    top_p = torch.tensor([0.9, 0.0, 1.0, float("nan"), 1.5])
    res = oracle.rejection_sample(tl, dl, ids, qi, ua, us, top_p=top_p)
    assert res.status == oracle.ERR_PARAM
    toks = res.out_tokens.view(B, 3)
    for r in (1, 3, 4):
        assert int(res.accepted_len[r]) == 0 and bool((toks[r] == -1).all())
    base = oracle.rejection_sample(tl, dl, ids, qi, ua, us)
    assert torch.equal(toks[2], base.out_tokens.view(B, 3)[2])       # top_p = 1 is the unfiltered rule
