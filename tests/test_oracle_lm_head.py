"""Pins for the oracle's LM head (CPU only): torch's float64 matmul on the widened inputs,
weights with known answers, linearity, and integer data whose result is exact in any precision."""
import numpy as np
import pytest
import torch

import oracle


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_against_torch_float64_matmul(dtype):
    g = torch.Generator().manual_seed(1)
    H = torch.randn(7, 96, generator=g).to(dtype)
    W = (torch.randn(53, 96, generator=g) / 10).to(dtype)
    ref = H.double() @ W.double().T
    got = oracle.lm_head(H, W)
    assert got.shape == (7, 53) and torch.allclose(got, ref, rtol=1e-13, atol=1e-13)
    part = oracle.lm_head(H, W, 10, 31)
    assert torch.equal(part, got[:, 10:31])                       # a column block is the same numbers


def test_known_weights_and_linearity():
    g = torch.Generator().manual_seed(2)
    H = torch.randn(5, 16, generator=g)
    eye = torch.eye(16)
    assert torch.equal(oracle.lm_head(H, eye), H.double())          # identity: logits = hidden states
    pick = torch.zeros(3, 16)
    pick[0, 4] = 1.0
    pick[1, 9] = -2.0                                                # transposed operands would not even have this shape
    out = oracle.lm_head(H, pick)
    assert torch.equal(out[:, 0], H[:, 4].double()) and torch.equal(out[:, 1], -2.0 * H[:, 9].double())
    assert float(out[:, 2].abs().max()) == 0.0
    W = torch.randn(11, 16, generator=g)
    a, b = oracle.lm_head(H, W), oracle.lm_head(2 * H, W)
    assert torch.equal(b, 2 * a)                                     # doubling is exact in binary
    with pytest.raises(oracle.OracleError):
        oracle.lm_head(H, W, 5, 12 + 5)


def test_integer_data_is_exact():
    rng = np.random.default_rng(3)
    H = torch.from_numpy(rng.integers(-2, 3, size=(9, 256)).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy(rng.integers(-1, 2, size=(40, 256)).astype(np.float32)).to(torch.bfloat16)
    got = oracle.lm_head(H, W)
    ref = (H.to(torch.int64) @ W.to(torch.int64).T).double()
    assert torch.equal(got, ref) and float(got.abs().max()) < 256   # representable in bf16 without rounding
