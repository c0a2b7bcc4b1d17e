"""Pins for the oracle's verification variants (per-request temperature, greedy), CPU only.

Checked against things other than the oracle: the output law at temperature tau (chi-square
against scipy's softmax of target/tau), a closed form (logits tau*ln(w) give p = w / sum w), the
exact invariance under scaling logits and temperature together by 2, numpy's argmax on rows with
ties, and the tau -> 0 limit, which must meet the separately coded greedy branch.
"""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

import oracle


def _uniforms(rng, n):
    return torch.from_numpy(rng.integers(0, 1 << 24, size=n).astype(np.float32) / float(1 << 24))


def _identical_requests(T, Dr, n_trials, tau, seed):
    rng = np.random.default_rng(seed)
    k, V = Dr.shape
    q = scipy.special.softmax(Dr.astype(np.float64) / tau, axis=1)
    ids = np.stack([rng.choice(V, size=n_trials, p=q[i]) for i in range(k)], axis=1)
    tl = torch.from_numpy(np.tile(T, (n_trials, 1)))
    dl = torch.from_numpy(np.tile(Dr, (n_trials, 1)))
    qi = torch.arange(0, (n_trials + 1) * (k + 1), k + 1, dtype=torch.int32)
    return tl, dl, torch.from_numpy(ids.reshape(-1).astype(np.int32)), qi, _uniforms(rng, n_trials * k), _uniforms(rng, n_trials)


@pytest.mark.parametrize("tau", [0.6, 2.5])
def test_output_law_at_temperature(tau):
    V, k, n_trials = 16, 2, 200_000
    rng = np.random.default_rng(int(tau * 10))
    T = (rng.standard_normal((k + 1, V)) * 1.5).astype(np.float32)
    Dr = (T[:k] + rng.standard_normal((k, V))).astype(np.float32)
    tl, dl, ids, qi, ua, us = _identical_requests(T, Dr, n_trials, tau, seed=3)
    res = oracle.rejection_sample(tl, dl, ids, qi, ua, us, temperature=torch.full((n_trials,), tau))
    p = scipy.special.softmax(T.astype(np.float64) / tau, axis=1)
    toks = res.out_tokens.view(n_trials, k + 1).numpy()
    hist0 = np.bincount(toks[:, 0], minlength=V)
    assert scipy.stats.chisquare(hist0, p[0] * n_trials).pvalue > 1e-3
    sel = res.accepted_len.numpy() >= 1
    hist1 = np.bincount(toks[sel, 1], minlength=V)
    assert scipy.stats.chisquare(hist1, p[1] * sel.sum()).pvalue > 1e-3
    # the temperature-1 law (tau ignored) and the inverse temperature (multiplied instead of divided) are rejected
    for wrong in (1.0, 1.0 / tau):
        pw = scipy.special.softmax(T[0].astype(np.float64) / wrong)
        assert scipy.stats.chisquare(hist0, pw * n_trials).pvalue < 1e-6
    # acceptance rate of the first draft: sum_v min(p, q) at this temperature
    q0 = scipy.special.softmax(Dr[0].astype(np.float64) / tau)
    beta = np.minimum(p[0], q0).sum()
    assert abs(sel.mean() - beta) < 5 * math.sqrt(beta * (1 - beta) / n_trials)


def test_softmax_closed_form_and_default():
    w = np.array([1.0, 2.0, 3.0, 4.0, 10.0])
    for tau in (0.5, 1.0, 3.0):
        row = torch.tensor(tau * np.log(w), dtype=torch.float32)
        p = oracle.softmax_row(row, tau=tau).numpy()
        assert np.allclose(p, w / w.sum(), rtol=1e-6)          # fp32 storage of the logits bounds the error
    row = torch.randn(100)
    assert torch.equal(oracle.softmax_row(row), oracle.softmax_row(row, tau=1.0))


def test_scaling_logits_and_temperature_by_two_changes_nothing():
    rng = np.random.default_rng(8)
    B, k, V = 40, 3, 50
    tl = torch.from_numpy(rng.standard_normal((B * (k + 1), V)).astype(np.float32))
    dl = tl.view(B, k + 1, V)[:, :k].reshape(B * k, V) + torch.from_numpy(rng.standard_normal((B * k, V)).astype(np.float32))
    ids = torch.from_numpy(rng.integers(0, V, size=B * k).astype(np.int32))
    qi = torch.arange(0, (B + 1) * (k + 1), k + 1, dtype=torch.int32)
    ua, us = _uniforms(rng, B * k), _uniforms(rng, B)
    tau = torch.from_numpy(rng.uniform(0.3, 2.0, size=B).astype(np.float32))
    a = oracle.rejection_sample(tl, dl, ids, qi, ua, us, temperature=tau)
    b = oracle.rejection_sample(tl * 2, dl * 2, ids, qi, ua, us, temperature=tau * 2)   # exact in binary
    assert torch.equal(a.accepted_len, b.accepted_len) and torch.equal(a.out_tokens, b.out_tokens)
    assert torch.equal(a.rho.nan_to_num(-1), b.rho.nan_to_num(-1))
    # and it is not the temperature-1 result
    c = oracle.rejection_sample(tl, dl, ids, qi, ua, us)
    assert not torch.equal(a.rho.nan_to_num(-1), c.rho.nan_to_num(-1))
    # temperature 1 given explicitly is the base rule, bit for bit
    d = oracle.rejection_sample(tl, dl, ids, qi, ua, us, temperature=torch.ones(B))
    assert torch.equal(c.out_tokens, d.out_tokens) and torch.equal(c.rho.nan_to_num(-1), d.rho.nan_to_num(-1))


def test_greedy_against_numpy_argmax_with_ties():
    rng = np.random.default_rng(21)
    B, k, V = 300, 4, 12
    # coarse integer logits: many ties for the maximum, so the lowest-id rule is exercised
    T = rng.integers(0, 4, size=(B, k + 1, V)).astype(np.float32)
    am = T.argmax(axis=2)                                     # numpy: first occurrence of the maximum
    ids = am[:, :k].copy()
    flip = rng.random((B, k)) < 0.3
    ids[flip] = rng.integers(0, V, size=int(flip.sum()))
    tl = torch.from_numpy(T.reshape(B * (k + 1), V))
    dl = torch.zeros((B * k, V))
    qi = torch.arange(0, (B + 1) * (k + 1), k + 1, dtype=torch.int32)
    res = oracle.rejection_sample(tl, dl, torch.from_numpy(ids.reshape(-1).astype(np.int32)), qi,
                                  torch.zeros(B * k), torch.zeros(B), temperature=torch.zeros(B))
    toks = res.out_tokens.view(B, k + 1).numpy()
    seen_tie_reject = False
    for r in range(B):
        match = ids[r] == am[r, :k]
        n = k if match.all() else int(np.argmin(match))
        assert int(res.accepted_len[r]) == n
        assert (toks[r, :n] == ids[r, :n]).all() and toks[r, n] == am[r, n] and (toks[r, n + 1:] == -1).all()
        if n < k and T[r, n, ids[r, n]] == T[r, n].max():
            seen_tie_reject = True                            # a draft that ties the maximum at a higher id is rejected
    assert seen_tie_reject
    assert oracle.argmax_row(torch.tensor([1.0, 5.0, 5.0, -2.0])) == 1


def test_small_temperature_meets_greedy_branch():
    rng = np.random.default_rng(33)
    B, k, V = 200, 3, 30
    T = rng.standard_normal((B, k + 1, V)).astype(np.float32)    # continuous: no ties, gaps far above 1e-3
    am = T.argmax(axis=2)
    ids = am[:, :k].copy()
    flip = rng.random((B, k)) < 0.3
    ids[flip] = rng.integers(0, V, size=int(flip.sum()))
    # a greedy draft: its own logits put all mass on the drafted token
    Dr = np.full((B, k, V), -50.0, dtype=np.float32)
    np.put_along_axis(Dr, ids[:, :, None], 50.0, axis=2)
    tl, dl = torch.from_numpy(T.reshape(-1, V)), torch.from_numpy(Dr.reshape(-1, V))
    qi = torch.arange(0, (B + 1) * (k + 1), k + 1, dtype=torch.int32)
    idt = torch.from_numpy(ids.reshape(-1).astype(np.int32))
    ua, us = _uniforms(rng, B * k), _uniforms(rng, B)
    greedy = oracle.rejection_sample(tl, dl, idt, qi, ua, us, temperature=torch.zeros(B))
    cold = oracle.rejection_sample(tl, dl, idt, qi, ua, us, temperature=torch.full((B,), 1e-4))
    top2 = np.sort(T, axis=2)
    clear = torch.from_numpy((top2[..., -1] - top2[..., -2]).min(axis=1) > 0.01)   # runner-up mass < e^-100
    same = (greedy.accepted_len == cold.accepted_len) & (greedy.out_tokens.view(B, -1) == cold.out_tokens.view(B, -1)).all(dim=1)
    assert int(clear.sum()) > B // 2 and bool(same[clear].all())
    assert int(greedy.accepted_len.sum()) not in (0, B * k)


def test_mixed_batch_and_bad_temperature():
    rng = np.random.default_rng(2)
    B, k, V = 6, 2, 20
    tl = torch.from_numpy(rng.standard_normal((B * (k + 1), V)).astype(np.float32))
    dl = torch.from_numpy(rng.standard_normal((B * k, V)).astype(np.float32))
    ids = torch.from_numpy(rng.integers(0, V, size=B * k).astype(np.int32))
    qi = torch.arange(0, (B + 1) * (k + 1), k + 1, dtype=torch.int32)
    ua, us = _uniforms(rng, B * k), _uniforms(rng, B)
    tau = torch.tensor([1.0, 0.0, 0.5, -1.0, float("nan"), 2.0])
    res = oracle.rejection_sample(tl, dl, ids, qi, ua, us, temperature=tau)
    assert res.status == oracle.ERR_PARAM
    toks = res.out_tokens.view(B, k + 1)
    for r in (3, 4):
        assert int(res.accepted_len[r]) == 0 and (toks[r] == -1).all()
    # every valid request equals the same request run alone at its temperature
    for r in (0, 1, 2, 5):
        one = oracle.rejection_sample(tl[r * 3:r * 3 + 3], dl[r * 2:r * 2 + 2], ids[r * 2:r * 2 + 2],
                                      torch.tensor([0, 3], dtype=torch.int32), ua[r * 2:r * 2 + 2], us[r:r + 1],
                                      temperature=tau[r:r + 1])
        assert torch.equal(one.out_tokens, toks[r]) and int(one.accepted_len[0]) == int(res.accepted_len[r])
