"""Pins for the oracle's restatement of the paper's scheduler numerics (CPU only): Eq. 1-4 with
Appendix A.1/A.2, the gain G of Section 5.2 with Appendix A.3, and Algorithm 1."""
import math

import numpy as np
import pytest
import scipy.stats
import torch

import oracle


@pytest.mark.parametrize("B,N,theta", [(64, 2, 0.7), (256, 4, 0.51), (100, 8, 0.79), (32, 3, 0.0), (32, 3, 1.0)])
def test_eq1_conserves_B_and_converges_to_eq2(B, N, theta):
    T = 4000
    sa, sr, n = oracle.sp_recurrence(B, N, theta, T)
    assert torch.allclose(sa + sr + n, torch.full((T + 1,), float(B), dtype=torch.float64), rtol=0, atol=1e-9)
    closed = oracle.sp_effective_batch(B, N, theta)
    assert math.isclose(closed, B / (N - theta * (N - 1)), rel_tol=1e-15)
    if theta > 0.0:       # theta = 0: the batch circulates with period N and does not converge
        assert math.isclose(float(sa[T] + n[T]), closed, rel_tol=1e-9)
    else:
        assert float((sa + n)[T - N + 1:].sum()) == pytest.approx(B)      # one burst of B per N iterations
    # first steps by hand: n_0 = B; s^a_1 = B theta; s^r_1 = B (1 - theta) for N >= 2
    assert float(sa[1]) == pytest.approx(B * theta) and float(sr[1]) == pytest.approx(B * (1 - theta) if N >= 2 else 0.0)
    if N >= 2:
        assert float(n[1]) == 0.0 and float(n[N]) == pytest.approx(B * (1 - theta))


def test_eq2_end_points():
    assert oracle.sp_effective_batch(128, 4, 1.0) == 128.0            # every speculation accepted: full batch
    assert oracle.sp_effective_batch(128, 4, 0.0) == 32.0             # none accepted: pipeline parallelism's B / N
    assert oracle.sp_effective_batch(128, 1, 0.3) == 128.0            # one stage: nothing in flight


@pytest.mark.parametrize("B,N,alpha", [(64, 2, 0.15), (256, 4, 0.3), (100, 8, 0.2), (50, 3, 0.0)])
def test_eq3_recurrence_converges_to_its_limit(B, N, alpha):
    T = 6000
    bt = oracle.alpha_recurrence(B, N, alpha, T)
    for i in range(N):
        assert float(bt[i]) == pytest.approx(B * (1 - alpha) ** i, rel=1e-14)
    closed = oracle.alpha_batch(B, N, alpha)
    assert math.isclose(closed, B / (1 + alpha * (N - 1)), rel_tol=1e-15)
    assert math.isclose(float(bt[T]), closed, rel_tol=1e-9)
    # the conserved quantity behind Appendix A.2's telescoping sum
    t = T - 5
    assert float(bt[t] + alpha * bt[t - N + 1:t].sum()) == pytest.approx(B, rel=1e-9)


def test_eq4_reduces_and_matches_hand_values():
    # alpha = 0: Eq. 4 is Eq. 2
    assert oracle.alpha_effective_batch(96, 4, 0.0, 0.6) == pytest.approx(oracle.sp_effective_batch(96, 4, 0.6), rel=1e-15)
    # hand value: B = 100, N = 2, alpha = 0.25, theta_alpha = 0.8: B_alpha = 80; 0.25*80 + 0.75*80/1.2 = 70
    assert oracle.alpha_batch(100, 2, 0.25) == pytest.approx(80.0, rel=1e-15)
    assert oracle.alpha_effective_batch(100, 2, 0.25, 0.8) == pytest.approx(70.0, rel=1e-14)
    # perfect accuracy: every sequence of the steady-state batch yields a token
    assert oracle.alpha_effective_batch(100, 4, 0.2, 1.0) == pytest.approx(oracle.alpha_batch(100, 4, 0.2), rel=1e-15)


def test_gain_equals_throughput_ratio_of_appendix_a3():
    rng = np.random.default_rng(0)
    for _ in range(20):
        I, n, bs = float(rng.integers(50, 500)), int(rng.integers(1, 5)), float(rng.integers(8, 256))
        t_d, t_p = rng.uniform(0.01, 0.05), rng.uniform(0.1, 1.0)
        i_wait = rng.integers(1, 20, size=n).astype(float)
        i_delay = float(rng.integers(1, 40))
        tok_aggr, T_aggr = (bs + 1) * I - i_wait.sum(), (I - (n + 1)) * t_d + (n + 1) * t_p
        tok_delay, T_delay = (bs + 1) * I - i_delay, (I - 1) * t_d + t_p
        ratio = (tok_delay / T_delay) / (tok_aggr / T_aggr)
        assert oracle.delay_gain(I, t_p / t_d, bs, i_delay, i_wait) == pytest.approx(ratio, rel=1e-12)
    # no recomputation penalty (pdr = 1) and equal waiting: no gain
    assert oracle.delay_gain(100, 1.0, 32, 7, [3, 4]) == pytest.approx(1.0, rel=1e-15)


def _algorithm1_bruteforce(ell, tau, prec, pp, theta, horizon):
    out = []
    for i in range(1, horizon + 1):
        terms = []
        for w in range(i // pp + 1):
            t = i - pp * w
            k = t + w
            terms.append((k, float(scipy.stats.binom.pmf(t, k, theta)) if k > 0 else 1.0))
        e_gen = sum(k * p for k, p in terms)
        p_fin = [prec[r] * sum(p for k, p in terms if k >= tau[r]) for r in range(len(ell))]
        out.append(sum(ell) + (len(ell) - sum(p_fin)) * e_gen - sum(l * p for l, p in zip(ell, p_fin)))
    return np.array(out)


@pytest.mark.parametrize("pp,theta", [(1, 0.7), (2, 0.51), (4, 0.79), (8, 0.6), (3, 0.0), (3, 1.0)])
def test_algorithm1_against_scipy_binomial_terms(pp, theta):
    rng = np.random.default_rng(pp)
    nreq = 37
    ell = rng.integers(10, 4000, size=nreq)
    tau = rng.choice([4, 8, 16, 32, 64, 10 ** 6], size=nreq)
    prec = rng.uniform(0.6, 0.95, size=nreq)
    M = oracle.lookahead_memory(torch.from_numpy(ell).int(), torch.from_numpy(tau).int(), torch.from_numpy(prec), pp, theta)
    ref = _algorithm1_bruteforce(ell.tolist(), tau.tolist(), prec.tolist(), pp, theta, 64)
    assert M.shape == (64,) and np.allclose(M.numpy(), ref, rtol=1e-11)


def test_algorithm1_closed_forms():
    ell = torch.tensor([100, 200, 300], dtype=torch.int32)
    tau = torch.tensor([4, 16, 1000], dtype=torch.int32)
    prec = torch.tensor([0.8, 0.9, 0.7], dtype=torch.float64)
    # pp = 1: k = i for every w and the terms are a full binomial law, so E[L_gen] = i and
    # P_fin = prec * [i >= tau];   theta = 1: only w = 0 survives, same result for any pp
    for pp, theta in ((1, 0.37), (5, 1.0)):
        M = oracle.lookahead_memory(ell, tau, prec, pp, theta)
        for i in range(1, 65):
            p_fin = [float(prec[r]) * (1.0 if i >= int(tau[r]) else 0.0) for r in range(3)]
            expect = 600 + (3 - sum(p_fin)) * i - sum(float(ell[r]) * p_fin[r] for r in range(3))
            assert float(M[i - 1]) == pytest.approx(expect, rel=1e-12), (pp, theta, i)
    # nobody finishes inside the window: memory grows by |B| E[L_gen]
    M = oracle.lookahead_memory(ell, torch.full((3,), 10 ** 6, dtype=torch.int32), prec, 1, 0.5)
    assert np.allclose(M.numpy(), 600 + 3 * np.arange(1, 65), rtol=1e-13)
    # an empty running set needs no memory
    e = torch.zeros(0, dtype=torch.int32)
    assert float(oracle.lookahead_memory(e, e, torch.zeros(0, dtype=torch.float64), 2, 0.5).abs().max()) == 0.0
