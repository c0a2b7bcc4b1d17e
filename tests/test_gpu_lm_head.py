"""GPU parity of the LM head against the oracle.

Floating-point data: |logit - oracle| <= 2^-8 |oracle| + 1e-3 (bf16 rounding of the result is
2^-9 relative; fp32 accumulation over K terms adds far less than the absolute term).  Integer
data whose products and sums are exact in every precision: bit-exact, which also lets the fused
statistics be checked through the sampling half against the oracle run on the oracle's own logits.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34370_b200 as spx

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _check_logits(H, W, cols=None):
    logits, stats, status = spx.lm_head(H.to(DEV), W.to(DEV))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    V = W.shape[0]
    got = logits[:, :V].float().cpu().double()
    if cols is None:
        ref = oracle.lm_head(H, W)
        err = (got - ref).abs()
        assert bool((err <= ref.abs() * 2.0 ** -8 + 1e-3).all()), float(err.max())
    else:
        for a, b in cols:
            ref = oracle.lm_head(H, W, a, b)
            err = (got[:, a:b] - ref).abs()
            assert bool((err <= ref.abs() * 2.0 ** -8 + 1e-3).all()), (a, b, float(err.max()))
    return logits, stats


@pytest.mark.parametrize("M,K,V", [(1, 64, 256), (7, 72, 100), (128, 512, 1024), (200, 520, 1000), (384, 1024, 5000)])
def test_small_shapes_match_oracle(M, K, V):
    g = torch.Generator().manual_seed(M + K + V)
    H = torch.randn(M, K, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, K, generator=g) / K ** 0.5).to(torch.bfloat16)
    logits, stats = _check_logits(H, W)
    # the statistics describe the stored values: recompute them from the same launch's logits on the host
    x = logits[:, :V].float().cpu().double()
    n_tiles = (V + 255) // 256
    for t in range(n_tiles):
        blk = x[:, t * 256:min(V, (t + 1) * 256)]
        mx = blk.max(dim=1).values
        s = torch.exp(blk - mx[:, None]).sum(dim=1)
        assert torch.allclose(stats[:, t, 0].cpu().double(), mx * 1.4426950408889634, rtol=1e-6, atol=1e-6)
        assert torch.allclose(stats[:, t, 1].cpu().double(), s, rtol=2e-5)


def test_integer_data_is_bit_exact_and_repeatable():
    rng = np.random.default_rng(5)
    M, K, V = 130, 448, 3000
    H = torch.from_numpy(rng.integers(-2, 3, size=(M, K)).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy((rng.integers(-1, 2, size=(V, K)) * (rng.random((V, K)) < 0.1)).astype(np.float32)).to(torch.bfloat16)
    ref = oracle.lm_head(H, W)
    assert float(ref.abs().max()) < 256
    logits, _, status = spx.lm_head(H.to(DEV), W.to(DEV))
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(logits[:, :V].float().cpu().double(), ref)
    for _ in range(3):
        again, _, _ = spx.lm_head(H.to(DEV), W.to(DEV))
        assert torch.equal(again[:, :V], logits[:, :V])


def test_llama_shape_on_sampled_column_blocks():
    g = torch.Generator().manual_seed(8)
    M, K, V = 384, 4096, 128256
    H = torch.randn(M, K, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, K, generator=g) * (3.0 / K ** 0.5)).to(torch.bfloat16)
    _check_logits(H, W, cols=[(0, 64), (2040, 2056), (65536 - 8, 65536 + 8), (V - 40, V)])


def test_bad_arguments():
    H = torch.zeros(4, 60, dtype=torch.bfloat16, device=DEV)       # hidden size not a multiple of 8
    W = torch.zeros(16, 60, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(spx.SpxError):
        spx.lm_head(H, W)
