"""Pins for the oracle's rejection-sampling half (CPU only).

Checked against things other than the oracle itself: the law of the emitted tokens (chi-square
against scipy's float64 softmax of the target rows, which is what speculative sampling must
reproduce), the exact identity min(p,q) + (1-beta) r/R = p, closed-form acceptance rates,
special cases with known answers, and a brute-force enumeration on tiny vocabularies against
numpy's searchsorted on directly built intervals.
"""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

import oracle


def _batch_of_identical_requests(T, Dr, n_trials, seed, dtype=torch.float32):
    """n_trials requests that all carry target rows T [k+1,V] and draft rows Dr [k,V].

    Draft ids are drawn from softmax(Dr) with numpy (harness side), uniforms on the 2^-24 grid.
    """
    rng = np.random.default_rng(seed)
    k, V = Dr.shape
    q = scipy.special.softmax(Dr.astype(np.float64), axis=1)
    ids = np.stack([rng.choice(V, size=n_trials, p=q[i]) for i in range(k)], axis=1) if k else \
        np.zeros((n_trials, 0), dtype=np.int64)
    tl = torch.from_numpy(np.tile(T, (n_trials, 1))).to(dtype)
    dl = torch.from_numpy(np.tile(Dr, (n_trials, 1))).to(dtype) if k else torch.zeros((0, V), dtype=dtype)
    q_indptr = torch.arange(0, (n_trials + 1) * (k + 1), k + 1, dtype=torch.int32)
    ua = torch.from_numpy(rng.integers(0, 1 << 24, size=n_trials * k).astype(np.float32) / float(1 << 24))
    us = torch.from_numpy(rng.integers(0, 1 << 24, size=n_trials).astype(np.float32) / float(1 << 24))
    return tl, dl, torch.from_numpy(ids.reshape(-1).astype(np.int32)), q_indptr, ua, us


@pytest.mark.parametrize("k", [1, 3])
def test_chi_square_output_law_is_target_law(k):
    V, n_trials = 16, 200_000
    rng = np.random.default_rng(100 + k)
    T = (rng.standard_normal((k + 1, V)) * 1.5).astype(np.float32)
    Dr = (T[:k] + rng.standard_normal((k, V)) * 1.0).astype(np.float32)
    tl, dl, ids, qi, ua, us = _batch_of_identical_requests(T, Dr, n_trials, seed=7 + k)
    res = oracle.rejection_sample(tl, dl, ids, qi, ua, us)
    p = scipy.special.softmax(T.astype(np.float64), axis=1)
    toks = res.out_tokens.view(n_trials, k + 1).numpy()
    n = res.accepted_len.numpy()
    # first emitted token ~ p_0
    hist0 = np.bincount(toks[:, 0], minlength=V)
    assert hist0.sum() == n_trials
    pv0 = scipy.stats.chisquare(hist0, p[0] * n_trials).pvalue
    assert pv0 > 1e-3, pv0
    # given the first draft was accepted, the second emitted token ~ p_1
    sel = n >= 1
    hist1 = np.bincount(toks[sel, 1], minlength=V)
    pv1 = scipy.stats.chisquare(hist1, p[1] * sel.sum()).pvalue
    assert pv1 > 1e-3, pv1
    # a wrong rule must be detectable at this sample size: the draft law is rejected
    q0 = scipy.special.softmax(Dr[0].astype(np.float64))
    assert scipy.stats.chisquare(hist0, q0 * n_trials).pvalue < 1e-6


def test_closed_form_acceptance_rates():
    V, k, n_trials = 16, 3, 200_000
    rng = np.random.default_rng(5)
    T = (rng.standard_normal((k + 1, V)) * 2.0).astype(np.float32)
    Dr = (T[:k] + rng.standard_normal((k, V))).astype(np.float32)
    tl, dl, ids, qi, ua, us = _batch_of_identical_requests(T, Dr, n_trials, seed=11)
    res = oracle.rejection_sample(tl, dl, ids, qi, ua, us)
    p = scipy.special.softmax(T.astype(np.float64), axis=1)
    q = scipy.special.softmax(Dr.astype(np.float64), axis=1)
    beta = np.minimum(p[:k], q).sum(axis=1)
    n = res.accepted_len.numpy()
    surv = 1.0
    for j in range(1, k + 1):
        surv *= beta[j - 1]                                  # P(n >= j) = prod_{i<j} beta_i
        emp = (n >= j).mean()
        sd = math.sqrt(surv * (1 - surv) / n_trials)
        assert abs(emp - surv) < 5 * sd, (j, emp, surv)


def test_residual_identity_reproduces_target():
    rng = np.random.default_rng(3)
    for V in (16, 1000):
        t = torch.from_numpy((rng.standard_normal(V) * 3).astype(np.float32))
        d = t + torch.from_numpy(rng.standard_normal(V).astype(np.float32))
        p, q = oracle.softmax_row(t), oracle.softmax_row(d)
        assert abs(float(p.sum()) - 1) < 1e-13 and abs(float(q.sum()) - 1) < 1e-13
        assert torch.allclose(p, torch.from_numpy(scipy.special.softmax(t.double().numpy())), rtol=1e-12)
        r, R = oracle.residual(p, q)
        beta = float(torch.minimum(p, q).sum())
        assert abs(R - (1 - beta)) < 1e-12
        assert torch.allclose(torch.minimum(p, q) + (1 - beta) * r / R, p, rtol=0, atol=1e-12)


def test_softmax_row_accepts_bf16():
    rng = np.random.default_rng(8)
    t = torch.from_numpy((rng.standard_normal(512) * 3).astype(np.float32)).to(torch.bfloat16)
    p = oracle.softmax_row(t)
    ref = scipy.special.softmax(t.double().numpy())
    assert np.allclose(p.numpy(), ref, rtol=1e-12)


def _run(T, Dr, ids, ua, us, dtype=torch.float32):
    """One request."""
    k = len(ids)
    tl = torch.tensor(T, dtype=dtype)
    dl = torch.tensor(Dr, dtype=dtype) if k else torch.zeros((0, tl.shape[1]), dtype=dtype)
    res = oracle.rejection_sample(tl, dl, torch.tensor(ids, dtype=torch.int32),
                                  torch.tensor([0, k + 1], dtype=torch.int32),
                                  torch.tensor(ua, dtype=torch.float32), torch.tensor([us], dtype=torch.float32))
    return int(res.accepted_len[0]), res.out_tokens.tolist(), res


def test_special_cases():
    rng = np.random.default_rng(21)
    V, k = 12, 3
    T = (rng.standard_normal((k + 1, V)) * 2).tolist()
    # q == p: every draft accepted whatever the uniforms, bonus from p_k
    n, toks, _ = _run(T, T[:k], [1, 5, 7], [0.999, 0.5, 0.0], 0.3)
    assert n == k and toks[:k] == [1, 5, 7]
    pk = scipy.special.softmax(np.array(T[k], dtype=np.float32).astype(np.float64))
    assert toks[k] == int(np.searchsorted(np.cumsum(pk), 0.3 * pk.sum(), side="right"))
    # a_i = 0 accepts everything when p(x) > 0
    Dr = (np.array(T[:k]) + rng.standard_normal((k, V))).tolist()
    n, toks, _ = _run(T, Dr, [0, 1, 2], [0.0, 0.0, 0.0], 0.9)
    assert n == k
    # disjoint supports: draft mass where the target has none -> reject at 0, resample from p_0
    Tdis = [[0.0 if v < 6 else -1e4 for v in range(V)]] * (k + 1)
    Ddis = [[-1e4 if v < 6 else 0.0 for v in range(V)]] * k
    for s, expect in ((0.0, 0), (0.49, 2), (0.51, 3), (1 - 2.0 ** -24, 5)):
        n, toks, res = _run(Tdis, Ddis, [8, 9, 10], [0.0, 0.0, 0.0], s)
        assert n == 0 and toks == [expect, -1, -1, -1], (s, toks)
        assert abs(float(res.resid_mass[0]) - 1.0) < 1e-12
    # one-hot target: the emitted token is that token whatever s
    Thot = [[-1e4] * V for _ in range(k + 1)]
    for row in Thot:
        row[4] = 0.0
    for s in (0.0, 0.37, 1 - 2.0 ** -24):
        n, toks, _ = _run(Thot, Dr, [3, 3, 3], [0.5, 0.5, 0.5], s)
        assert n == 0 and toks[0] == 4
    # k = 0: plain sampling from p_0
    n, toks, _ = _run([T[0]], [], [], [], 0.62)
    p0 = scipy.special.softmax(np.array(T[0], dtype=np.float32).astype(np.float64))
    assert n == 0 and toks == [int(np.searchsorted(np.cumsum(p0), 0.62 * p0.sum(), side="right"))]
    # s = 0 picks the first token with positive residual; s -> 1 the last one
    p0 = scipy.special.softmax(np.array(T[0], dtype=np.float32).astype(np.float64))
    q0 = scipy.special.softmax(np.array(Dr[0], dtype=np.float32).astype(np.float64))
    pos = np.nonzero(p0 - q0 > 0)[0]
    xrej = int(np.argmax(q0 / p0))                          # p/q smallest here
    rho = p0[xrej] / q0[xrej]
    assert rho < 0.99
    n, toks, _ = _run(T, Dr, [xrej, 0, 0], [0.995, 0.0, 0.0], 0.0)
    assert n == 0 and toks[0] == pos[0]
    n, toks, _ = _run(T, Dr, [xrej, 0, 0], [0.995, 0.0, 0.0], 1 - 2.0 ** -24)
    assert n == 0 and toks[0] == pos[-1]


def test_accept_threshold_is_strict_ratio():
    # p(x)/q(x) is a known number: accept iff a < p/q.
    V = 4
    T = [[math.log(1), math.log(2), math.log(3), math.log(4)]] * 2        # p = .1 .2 .3 .4
    Dr = [[math.log(4), math.log(3), math.log(2), math.log(1)]]           # q = .4 .3 .2 .1
    # x = 0: rho = 0.25
    n, _, res = _run(T, Dr, [0], [0.2499], 0.5)
    assert n == 1 and abs(float(res.rho[0]) - 0.25) < 1e-6
    n, _, _ = _run(T, Dr, [0], [0.2501], 0.5)
    assert n == 0
    # x = 3: rho = 4 > 1 always accepts
    n, _, _ = _run(T, Dr, [3], [1 - 2.0 ** -24], 0.5)
    assert n == 1
    # residual = max(0,p-q) = (0,0,.1,.3)/.4 : s < .25 -> token 2, else token 3
    for s, tok in ((0.0, 2), (0.2499, 2), (0.2501, 3), (0.99, 3)):
        n, toks, res = _run(T, Dr, [0], [0.9], s)
        assert n == 0 and toks[0] == tok
        assert abs(float(res.resid_mass[0]) - 0.4) < 1e-6


def test_brute_force_tiny_vocab_grid():
    rng = np.random.default_rng(77)
    for V in (3, 5, 8):
        for k in (1, 2):
            T = (rng.standard_normal((k + 1, V)) * 1.5).astype(np.float32)
            Dr = (T[:k] + rng.standard_normal((k, V))).astype(np.float32)
            p = scipy.special.softmax(T.astype(np.float64), axis=1)
            q = scipy.special.softmax(Dr.astype(np.float64), axis=1)
            grid = (np.arange(0, 1 << 24, (1 << 24) // 13)).astype(np.float32) / float(1 << 24)
            for ids in np.ndindex(*([V] * k)):
                for a in np.ndindex(*([len(grid)] * k)):
                    ua = [float(grid[i]) for i in a]
                    for s in grid[::3]:
                        # direct interval arithmetic
                        n_exp = k
                        for i in range(k):
                            if not (ua[i] < p[i, ids[i]] / q[i, ids[i]]):
                                n_exp = i
                                break
                        dist = np.maximum(p[n_exp] - q[n_exp], 0) if n_exp < k else p[k]
                        edges = np.cumsum(dist)
                        y_exp = int(np.searchsorted(edges, float(s) * edges[-1], side="right"))
                        ratios = [p[i, ids[i]] / q[i, ids[i]] for i in range(k)]
                        if min(abs(r - u) for r, u in zip(ratios, ua)) < 1e-9:
                            continue
                        if np.min(np.abs(edges - float(s) * edges[-1])) < 1e-12:
                            continue
                        n, toks, _ = _run(T.tolist(), Dr.tolist(), list(ids), ua, float(s))
                        assert n == n_exp and toks[n] == y_exp, (V, k, ids, ua, s)
                        assert toks[:n] == list(ids[:n]) and all(t == -1 for t in toks[n + 1:])
            if V >= 5:
                break        # k = 2 only for the smallest vocabularies (keeps the test fast)


def test_rows_after_first_rejection_are_never_consulted():
    rng = np.random.default_rng(9)
    V, k = 32, 4
    T = (rng.standard_normal((k + 1, V)) * 2).astype(np.float32)
    Dr = (T[:k] + rng.standard_normal((k, V))).astype(np.float32)
    p0 = scipy.special.softmax(T[1].astype(np.float64))
    q0 = scipy.special.softmax(Dr[1].astype(np.float64))
    xrej = int(np.argmax(q0 / p0))
    ids = [int(np.argmax(T[0] - Dr[0])), xrej, 3, 4]            # accept 0 (rho>=1), reject 1
    n, toks, _ = _run(T.tolist(), Dr.tolist(), ids, [0.5, 0.999, 0.1, 0.1], 0.4)
    assert n == 1
    T2, D2 = T.copy(), Dr.copy()
    T2[2:] = rng.standard_normal((k - 1, V))
    D2[2:] = rng.standard_normal((k - 2, V))
    n2, toks2, _ = _run(T2.tolist(), D2.tolist(), ids[:2] + [0, 0], [0.5, 0.999, 0.9, 0.9], 0.4)
    assert (n2, toks2) == (n, toks)


def test_invalid_draft_id_is_reported_and_isolated():
    V = 8
    T = np.zeros((2, V), dtype=np.float32).tolist()
    tl = torch.tensor(T * 2)
    dl = torch.tensor([T[0]] * 2)
    res = oracle.rejection_sample(tl, dl, torch.tensor([V, 1], dtype=torch.int32),
                                  torch.tensor([0, 2, 4], dtype=torch.int32),
                                  torch.tensor([0.5, 0.5]), torch.tensor([0.1, 0.1]))
    assert res.status == oracle.ERR_TOKEN
    assert res.accepted_len.tolist() == [0, 1] and res.out_tokens.tolist()[:2] == [-1, -1]
    assert res.out_tokens.tolist()[2] == 1 and res.out_tokens.tolist()[3] == 0


def test_emit_cdf_brackets_the_emitted_token():
    import spx_workloads as W
    b = W.generate(W.CONFIGS[0])
    res = oracle.rejection_sample(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept,
                                  b.u_sample)
    for r in range(b.batch):
        n = int(res.accepted_len[r])
        y = int(res.out_tokens[int(b.q_indptr[r]) + n])
        cdf, R = oracle.emit_cdf(r, n, b.target_logits, b.draft_logits, b.q_indptr)
        target = float(b.u_sample[r]) * R
        lo = float(cdf[y - 1]) if y > 0 else 0.0
        assert lo <= target < float(cdf[y])
        assert abs(R - float(res.resid_mass[r])) < 1e-15
        assert float(res.cdf_lo[r]) == lo and float(res.cdf_hi[r]) == float(cdf[y])
