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
from paper_2609_34370_b200 import binding

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


@pytest.mark.parametrize("M,K,V", [(1, 64, 256), (7, 72, 100), (128, 512, 1024), (200, 520, 1000), (384, 1024, 5000), (300, 256, 700), (520, 128, 900)])
def test_small_shapes_match_oracle(M, K, V):
    g = torch.Generator().manual_seed(M + K + V)
    H = torch.randn(M, K, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, K, generator=g) / K ** 0.5).to(torch.bfloat16)
    logits, stats = _check_logits(H, W)
    # the statistics describe the stored values: recompute them from the same launch's logits on the host
    x = logits[:, :V].float().cpu().double()
    cols = binding.LM_TILE_COLS
    n_tiles = (V + cols - 1) // cols
    assert stats.shape[1] == n_tiles
    for t in range(n_tiles):
        blk = x[:, t * cols:min(V, (t + 1) * cols)]
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


def test_fused_statistics_feed_the_sampling_half():
    """Integer data: the GPU's logits equal the oracle's bit for bit, so the sampling half run on them with
    the epilogue's statistics can be held against the oracle run on the oracle's own logits."""
    from parity_util import check_sampling
    rng = np.random.default_rng(11)
    B, k, K, V = 24, 3, 64, 5000
    TQ, TD = B * (k + 1), B * k
    H = torch.from_numpy(rng.integers(-2, 3, size=(TQ, K)).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy((rng.integers(-1, 2, size=(V, K)) * (rng.random((V, K)) < 0.3)).astype(np.float32)).to(torch.bfloat16)
    ref_logits = oracle.lm_head(H, W)
    assert float(ref_logits.abs().max()) < 256
    T = ref_logits.to(torch.bfloat16)                               # exact
    qi = torch.arange(0, (B + 1) * (k + 1), k + 1, dtype=torch.int32)
    t_rows = torch.tensor([r * (k + 1) + i for r in range(B) for i in range(k)])
    Dr = (T[t_rows].float() + torch.from_numpy(rng.integers(-1, 2, size=(TD, V)).astype(np.float32))).to(torch.bfloat16)
    g = torch.Generator().manual_seed(3)
    ids = torch.multinomial(torch.softmax(Dr.float(), dim=1), 1, generator=g).view(-1).to(torch.int32)
    ua, us = torch.rand(TD, generator=g), torch.rand(B, generator=g)
    logits, stats, status = spx.lm_head(H.to(DEV), W.to(DEV))
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(logits[:, :V].cpu(), T)
    acc, tok, _, ws = spx.rejection_sample(logits, Dr.to(DEV).contiguous(), ids.to(DEV), qi.to(DEV), ua.to(DEV), us.to(DEV),
                                           vocab=V, target_tile_stats=stats)
    acc0, tok0, _, _ = spx.rejection_sample(logits, Dr.to(DEV).contiguous(), ids.to(DEV), qi.to(DEV), ua.to(DEV), us.to(DEV), vocab=V)
    torch.cuda.synchronize()
    assert int(ws.status.item()) == 0

    class _B:
        pass
    bb = _B()
    bb.batch, bb.q_indptr, bb.u_accept, bb.u_sample = B, qi, ua, us
    bb.target_logits, bb.draft_logits, bb.draft_ids = T, Dr, ids
    bb.spec = type("S", (), {"vocab": V})
    rep = check_sampling(bb, acc, tok)
    assert not rep.hard_mismatch, rep
    assert int(acc.sum()) > 0
    print(f"\n[fused statistics] exact {rep.exact}/{rep.requests}, near ties {rep.accept_near_tie + rep.cdf_near_tie}; "
          f"same as the unfused pass on {int((acc == acc0).sum())}/{B} requests")


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
