"""GPU parity of the selective-speculation support calls against the oracle.

Confidence: fp32 results of fp32 partial sums merged in float64 against a float64 softmax;
tolerance 1e-5 relative (observed ~1e-6: the approximate exp2 is good to 2 ulp and the sums
average the per-term rounding).  Selection: integer-exact on identical stored inputs.
"""
import numpy as np
import pytest
import torch

import oracle
import spx_workloads as W
import paper_2609_34370_b200 as spx

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
CONF_RTOL = 1e-5


def _check_conf(b_cpu, vocab=None):
    b = b_cpu.to(DEV)
    cmax, ctok, creq, ws = spx.draft_confidence(b.draft_logits, b.draft_ids, b.q_indptr, vocab=vocab)
    torch.cuda.synchronize()
    assert int(ws.status.item()) == 0
    rmax, rtok, rreq = oracle.draft_confidence(b_cpu.draft_logits, b_cpu.draft_ids, b_cpu.q_indptr, vocab=vocab)
    worst = 0.0
    for g, r in ((cmax, rmax), (ctok, rtok), (creq, rreq)):
        if r.numel() == 0:
            continue
        rel = ((g.cpu().double() - r).abs() / r.clamp_min(1e-300))
        # probabilities below fp32's normal range are compared absolutely
        ok = (rel <= CONF_RTOL) | ((g.cpu().double() - r).abs() <= 1e-37)
        assert bool(ok.all()), float(rel.max())
        worst = max(worst, float(rel[r > 1e-30].max()) if bool((r > 1e-30).any()) else 0.0)
    return worst, rreq


@pytest.mark.parametrize("idx,vocab", [(0, None), (1, 5000), (1, 128256), (4, 40000)])
def test_confidence_matches_oracle(idx, vocab):
    spec = W.CONFIGS[idx] if idx == 0 else W.scaled(W.CONFIGS[idx], batch=16, ctx_div=64, vocab=vocab)
    worst, _ = _check_conf(W.generate(spec))
    print(f"\n[{spec.name} V={spec.vocab}] worst relative error of the confidences {worst:.2e}")


def test_confidence_full_size_ragged_vocab_and_bad_id():
    worst, _ = _check_conf(W.generate(W.CONFIGS[1]))
    print(f"\n[llama3-8b] worst relative error of the confidences {worst:.2e}")
    # ragged vocabulary inside a padded row (padding holds poison), k = 0 requests in the batch
    V, VS = 777, 784
    g = torch.Generator().manual_seed(3)
    qi = torch.tensor([0, 3, 4, 8, 9], dtype=torch.int32)             # k = 2, 0, 3, 0
    dl = torch.full((5, VS), 1e4, dtype=torch.bfloat16)
    dl[:, :V] = (torch.randn(5, V, generator=g) * 3).to(torch.bfloat16)
    ids = torch.tensor([1, 776, 5, 6, 7], dtype=torch.int32)
    cmax, ctok, creq, ws = spx.draft_confidence(dl.to(DEV), ids.to(DEV), qi.to(DEV), vocab=V)
    torch.cuda.synchronize()
    rmax, rtok, rreq = oracle.draft_confidence(dl, ids, qi, vocab=V)
    assert int(ws.status.item()) == 0
    assert torch.allclose(cmax.cpu().double(), rmax, rtol=CONF_RTOL) and torch.allclose(ctok.cpu().double(), rtok, rtol=CONF_RTOL)
    assert torch.allclose(creq.cpu().double(), rreq, rtol=CONF_RTOL) and float(creq[1]) == 1.0 and float(creq[3]) == 1.0
    ids[1] = V                                                        # first id past the vocabulary
    cmax2, ctok2, _, ws = spx.draft_confidence(dl.to(DEV), ids.to(DEV), qi.to(DEV), vocab=V)
    torch.cuda.synchronize()
    assert int(ws.status.item()) == spx.DEV_BAD_TOKEN
    assert torch.equal(cmax2, cmax) and bool(torch.isnan(ctok2[1])) and float(ctok2[0]) == float(ctok[0])


@pytest.mark.parametrize("B", [1, 7, 64, 257, 1024, 1025, 5000, 40000])
def test_selection_is_integer_exact(B):
    rng = np.random.default_rng(B)
    conf = rng.random(B).astype(np.float32)
    conf[rng.integers(0, B, size=B // 3)] = 0.5                       # many ties, also at the threshold
    k_in = rng.integers(0, 4, size=B).astype(np.int32)
    conf_t, k_t = torch.from_numpy(conf), torch.from_numpy(k_in)
    for alpha in (0.0, 0.15, 0.3, 0.5, 1.0):
        k_out, n_drop, status = spx.select_speculation(conf_t.to(DEV), k_t.to(DEV), alpha)
        torch.cuda.synchronize()
        ref, ref_drop = oracle.select_speculation(conf_t, k_t, alpha)
        assert int(status.item()) == 0 and int(n_drop.item()) == ref_drop
        assert torch.equal(k_out.cpu(), ref), (B, alpha)


def test_selection_special_values_aliasing_and_faults():
    conf = torch.tensor([0.0, -0.0, float("inf"), float("nan"), 1.0, 0.25, 0.25, 0.25, 0.25])
    k_in = torch.tensor([1, 1, 1, 1, 1, 2, 2, 2, 2], dtype=torch.int32)
    for alpha in (0.25, 0.45, 0.7, 0.9):
        ref, _ = oracle.select_speculation(conf, k_in, alpha)
        k_dev = k_in.to(DEV)
        out, _, status = spx.select_speculation(conf.to(DEV), k_dev, alpha, out=k_dev)     # in place
        torch.cuda.synchronize()
        assert int(status.item()) == 0 and torch.equal(out.cpu(), ref), alpha
    # all confidences equal: the highest indices go
    out, n_drop, _ = spx.select_speculation(torch.full((10,), 0.3, device=DEV), torch.full((10,), 3, dtype=torch.int32, device=DEV), 0.35)
    assert int(n_drop.item()) == 3 and out.cpu().tolist() == [3] * 7 + [0] * 3
    # a negative k is reported and treated as "no drafts"
    bad = torch.tensor([2, -1, 2, 2], dtype=torch.int32, device=DEV)
    out, n_drop, status = spx.select_speculation(torch.tensor([0.9, 0.1, 0.2, 0.5], device=DEV), bad, 0.34)
    torch.cuda.synchronize()
    assert int(status.item()) == spx.DEV_BAD_LEN and out.cpu().tolist() == [2, 0, 0, 2] and int(n_drop.item()) == 1
    with pytest.raises(spx.SpxError):
        spx.select_speculation(torch.zeros(3, device=DEV), torch.ones(3, dtype=torch.int32, device=DEV), 1.01)


def test_confidence_then_selection_on_the_selective_mix_workload():
    spec = W.scaled(W.CONFIGS[4], batch=64, ctx_div=64, vocab=32000)
    b_cpu = W.generate(spec)
    _, rreq = _check_conf(b_cpu)
    k_in = torch.tensor(b_cpu.k_host, dtype=torch.int32)
    conf32 = rreq.float()                                             # the oracle's confidences, stored as fp32, feed both sides
    for alpha in (0.15, 0.3):
        ref, ref_drop = oracle.select_speculation(conf32, k_in, alpha)
        out, n_drop, status = spx.select_speculation(conf32.to(DEV), k_in.to(DEV), alpha)
        torch.cuda.synchronize()
        assert int(status.item()) == 0 and int(n_drop.item()) == ref_drop and torch.equal(out.cpu(), ref)
        assert int((ref > 0).sum()) == int((k_in > 0).sum()) - ref_drop
