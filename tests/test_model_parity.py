"""Parity of the library's scheduler numerics with the oracle: Algorithm 1 on the GPU (float64 on
both sides, sums in a different order: 1e-12 relative), the scalar closed forms on the host."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34370_b200 as spx

DEV = "cuda:0"


@pytest.mark.gpu
@pytest.mark.parametrize("pp,theta", [(1, 0.7), (2, 0.51), (4, 0.79), (8, 0.6), (3, 0.0), (3, 1.0), (64, 0.5), (100, 0.5)])
@pytest.mark.parametrize("nreq", [0, 1, 37, 5000])
def test_lookahead_memory_matches_oracle(pp, theta, nreq):
    rng = np.random.default_rng(pp * 1000 + nreq)
    ell = torch.from_numpy(rng.integers(10, 8192, size=nreq).astype(np.int32))
    tau = torch.from_numpy(rng.choice([1, 4, 8, 16, 32, 64, 65, 10 ** 6], size=nreq).astype(np.int32))
    prec = torch.from_numpy(rng.uniform(0.5, 1.0, size=nreq))
    ref = oracle.lookahead_memory(ell, tau, prec, pp, theta)
    got = spx.lookahead_memory(ell.to(DEV), tau.to(DEV), prec.to(DEV), pp, theta)
    torch.cuda.synchronize()
    assert got.shape == (64,)
    assert torch.allclose(got.cpu(), ref, rtol=1e-12, atol=1e-9), float((got.cpu() - ref).abs().max())
    if nreq:
        h = spx.lookahead_memory(ell.to(DEV), tau.to(DEV), prec.to(DEV), pp, theta, horizon=200)
        assert torch.allclose(h.cpu(), oracle.lookahead_memory(ell, tau, prec, pp, theta, horizon=200), rtol=1e-12, atol=1e-9)


@pytest.mark.gpu
def test_lookahead_rejects_bad_arguments():
    z = torch.zeros(4, dtype=torch.int32, device=DEV)
    p = torch.ones(4, dtype=torch.float64, device=DEV)
    for kw in (dict(pp=0, theta=0.5), dict(pp=2, theta=1.5), dict(pp=2, theta=0.5, horizon=0), dict(pp=2, theta=0.5, horizon=257)):
        with pytest.raises(spx.SpxError):
            spx.lookahead_memory(z, z, p, **kw)


def test_closed_forms_match_oracle_on_the_host():
    rng = np.random.default_rng(1)
    for _ in range(50):
        B, N = float(rng.integers(1, 512)), int(rng.integers(1, 9))
        theta, alpha = float(rng.uniform(0, 1)), float(rng.uniform(0, 0.5))
        assert spx.sp_effective_batch(B, N, theta) == pytest.approx(oracle.sp_effective_batch(B, N, theta), rel=1e-15)
        assert spx.selective_batch(B, N, alpha) == pytest.approx(oracle.alpha_batch(B, N, alpha), rel=1e-15)
        assert spx.selective_effective_batch(B, N, alpha, theta) == pytest.approx(
            oracle.alpha_effective_batch(B, N, alpha, theta), rel=1e-14)
        n = int(rng.integers(1, 5))
        wait = rng.integers(1, 20, size=n).astype(float).tolist()
        args = (float(rng.integers(50, 500)), float(rng.uniform(2, 40)), float(rng.integers(8, 256)), float(rng.integers(1, 40)))
        assert spx.delay_gain(*args, wait) == pytest.approx(oracle.delay_gain(*args, wait), rel=1e-14)
