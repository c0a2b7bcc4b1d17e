"""GPU parity of the verification variants (per-request temperature, greedy) against the oracle.

Sampled requests: bit-exact (accepted_len, out_tokens) outside the two counted near-tie classes of
the base rule.  Greedy requests: bit-exact with no exemption (an argmax over stored values).
"""
import dataclasses

import pytest
import torch

import oracle
import spx_workloads as W
import paper_2609_34370_b200 as spx
from parity_util import check_sampling

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TAUS = [1.0, 0.0, 0.3, 0.7, 0.0, 1.5, 4.0, 0.05]


def _mixed_temperature(batch):
    return torch.tensor([TAUS[r % len(TAUS)] for r in range(batch)], dtype=torch.float32)


def _steer_greedy_drafts(b_cpu, tau, seed):
    """Harness side: for greedy requests, replace most draft ids with the target row's argmax (torch's)
    so that chains of greedy acceptances occur; the oracle still decides what is expected."""
    g = torch.Generator().manual_seed(seed)
    ids = b_cpu.draft_ids.clone()
    qi = b_cpu.q_indptr.tolist()
    for r in range(b_cpu.batch):
        if float(tau[r]) != 0.0:
            continue
        t0, k = qi[r], qi[r + 1] - qi[r] - 1
        for i in range(k):
            if torch.rand((), generator=g) < 0.8:
                ids[t0 - r + i] = int(torch.argmax(b_cpu.target_logits[t0 + i, :b_cpu.spec.vocab].float()))
    return dataclasses.replace(b_cpu, draft_ids=ids)


def _run(b_cpu, tau, **kw):
    b = b_cpu.to(DEV)
    acc, tok, ratio, ws = spx.rejection_sample(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept,
                                               b.u_sample, temperature=tau.to(DEV), **kw)
    torch.cuda.synchronize()
    return acc, tok, ratio, ws


@pytest.mark.parametrize("idx,vocab", [(0, None), (1, 5000), (1, 128256), (4, 40000)])
def test_mixed_temperatures_match_oracle(idx, vocab):
    spec = W.CONFIGS[idx] if idx == 0 else W.scaled(W.CONFIGS[idx], batch=16, ctx_div=64, vocab=vocab)
    b_cpu = W.generate(spec)
    tau = _mixed_temperature(b_cpu.batch)
    b_cpu = _steer_greedy_drafts(b_cpu, tau, seed=idx)
    acc, tok, ratio, ws = _run(b_cpu, tau, want_ratio=True)
    assert int(ws.status.item()) == 0
    ref = oracle.rejection_sample(b_cpu.target_logits, b_cpu.draft_logits, b_cpu.draft_ids, b_cpu.q_indptr,
                                  b_cpu.u_accept, b_cpu.u_sample, temperature=tau)
    rep = check_sampling(b_cpu, acc, tok, ref, temperature=tau)
    assert not rep.hard_mismatch, rep
    print(f"\n[{spec.name} V={spec.vocab}] exact {rep.exact}/{rep.requests}, accept-near-tie {rep.accept_near_tie}, "
          f"cdf-near-tie {rep.cdf_near_tie}, cdf-abs-near-tie {rep.cdf_abs_near_tie}")
    greedy = [r for r in range(b_cpu.batch) if float(tau[r]) == 0.0]
    assert sum(int(ref.accepted_len[r]) for r in greedy) > 0          # acceptance chains were exercised
    # the reported ratios agree with the oracle's where both consulted the draft
    both = torch.isfinite(ref.rho) & torch.isfinite(ratio.cpu().double()) & (ref.rho < 1e6)
    if bool(both.any()):
        rel = ((ratio.cpu().double() - ref.rho).abs() / ref.rho.clamp_min(1e-30))[both]
        assert float(rel.max()) < 2e-5, float(rel.max())


def test_temperature_one_equals_base_rule_and_bad_values_are_reported():
    spec = W.scaled(W.CONFIGS[1], batch=12, ctx_div=64, vocab=20000)
    b_cpu = W.generate(spec)
    b = b_cpu.to(DEV)
    acc0, tok0, _, _ = spx.rejection_sample(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample)
    acc1, tok1, _, ws = _run(b_cpu, torch.ones(b_cpu.batch))
    assert int(ws.status.item()) == 0
    rep = check_sampling(b_cpu, acc1, tok1, temperature=torch.ones(b_cpu.batch))
    assert not rep.hard_mismatch
    assert torch.equal(acc0, acc1) or rep.accept_near_tie + rep.cdf_near_tie > 0
    tau = torch.ones(b_cpu.batch)
    tau[2], tau[5], tau[7] = -0.5, float("nan"), float("inf")
    acc, tok, _, ws = _run(b_cpu, tau)
    assert int(ws.status.item()) == spx.DEV_BAD_PARAM
    qi = b_cpu.q_indptr.tolist()
    for r in range(b_cpu.batch):
        if r in (2, 5, 7):
            assert int(acc[r]) == 0 and bool((tok[qi[r]:qi[r + 1]] == -1).all())
        else:
            assert int(acc[r]) == int(acc1[r]) and torch.equal(tok[qi[r]:qi[r + 1]], tok1[qi[r]:qi[r + 1]])


def test_greedy_ties_across_and_inside_sub_segments():
    V, k = 70001, 3                                   # ragged tail: the last sub-segment holds 369 tokens
    g = torch.Generator().manual_seed(12)
    B = 6
    VS = 70008                                        # row stride: a multiple of 16 bytes; the padding holds poison
    T = (torch.randn(B * (k + 1), VS, generator=g) * 2).to(torch.bfloat16)
    T[:, V:] = 1e4
    Dr = torch.zeros(B * k, VS, dtype=torch.bfloat16)
    qi = torch.arange(0, (B + 1) * (k + 1), k + 1, dtype=torch.int32)
    big = 40.0
    ties = {0: (5000, 69000), 1: (100, 101), 2: (2047, 2048), 3: (70000, 70000), 4: (0, 70000), 5: (33333, 33334)}
    ids = torch.zeros(B * k, dtype=torch.int32)
    for r, (lo, hi) in ties.items():
        for i in range(k + 1):
            T[r * (k + 1) + i, lo] = big
            T[r * (k + 1) + i, hi] = big
        # drafts: lowest id (accepted), lowest id again, then the higher id of the tie (rejected unless lo == hi)
        ids[r * k:(r + 1) * k] = torch.tensor([lo, lo, hi])
    tau = torch.zeros(B)
    ref = oracle.rejection_sample(T, Dr, ids, qi, torch.zeros(B * k), torch.zeros(B), vocab=V, temperature=tau)
    acc, tok, _, ws = spx.rejection_sample(T.to(DEV), Dr.to(DEV), ids.to(DEV), qi.to(DEV), torch.zeros(B * k, device=DEV),
                                           torch.zeros(B, device=DEV), vocab=V, temperature=tau.to(DEV))
    torch.cuda.synchronize()
    assert int(ws.status.item()) == 0
    assert ref.accepted_len.tolist() == [2, 2, 2, 3, 2, 2]
    assert torch.equal(acc.cpu(), ref.accepted_len) and torch.equal(tok.cpu(), ref.out_tokens)


def test_full_size_mixed_temperatures():
    spec = W.CONFIGS[1]
    b_cpu = W.generate(spec)
    tau = _mixed_temperature(b_cpu.batch)
    b_cpu = _steer_greedy_drafts(b_cpu, tau, seed=1)
    acc, tok, _, ws = _run(b_cpu, tau)
    assert int(ws.status.item()) == 0
    rep = check_sampling(b_cpu, acc, tok, temperature=tau)
    assert not rep.hard_mismatch, rep
    print(f"\n[{spec.name}, mixed temperatures] exact {rep.exact}/{rep.requests}, accept-near-tie {rep.accept_near_tie}, "
          f"cdf-near-tie {rep.cdf_near_tie}, cdf-abs-near-tie {rep.cdf_abs_near_tie}")
    # the whole step takes the variant too, and agrees with the sampling half run alone
    b = b_cpu.to(DEV)
    out = torch.empty_like(b.q)
    lse = torch.empty(b.q.shape[:2], dtype=torch.float32, device=DEV)
    acc2, tok2 = torch.empty_like(acc), torch.empty_like(tok)
    a = spx.make_attn_args(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                           spec.num_kv_heads, spec.page_size, b.num_pages, out, lse, 0.0, max(b.k_host) + 1)
    tau_d = tau.to(DEV)
    s = spx.make_sample_args(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample, acc2, tok2,
                             None, None, tau_d)
    ws2 = spx.Workspace.allocate(spx.workspace_size(a, s), DEV)
    spx.verify_step(a, s, ws2, DEV)
    torch.cuda.synchronize()
    assert int(ws2.status.item()) == 0
    assert torch.equal(acc2, acc) and torch.equal(tok2, tok)
