"""GPU parity of top-k / top-p filtered verification against the oracle.

Bit-exact (accepted_len, out_tokens) outside the counted near-tie classes of parity_util (accept
band, CDF bands, and the top-p crossing band).  top-k alone involves no floating-point decision.
"""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
import spx_workloads as W
import paper_2609_34370_b200 as spx
from parity_util import check_sampling

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOP_K = [0, 50, 1, 0, 1000, 5, 0, 20]
TOP_P = [1.0, 1.0, 1.0, 0.9, 0.95, 0.5, 0.3, 1.0]
TAUS = [1.0, 0.7, 1.0, 1.0, 1.3, 0.8, 0.0, 1.0]


def _params(batch, vocab):
    tk = torch.tensor([TOP_K[r % 8] for r in range(batch)], dtype=torch.int32)
    tp = torch.tensor([TOP_P[r % 8] for r in range(batch)], dtype=torch.float32)
    tau = torch.tensor([TAUS[r % 8] for r in range(batch)], dtype=torch.float32)
    return tau, tk, tp


def _redraft(b_cpu, tau, tk, tp, seed):
    """Harness side: redraw the draft ids from the FILTERED draft distribution (the oracle's own
    filtered rows serve as the generator's law; the expectation still comes from the full oracle
    run), so that acceptance chains occur under filtering.  A few ids are left as they were, which
    exercises drafts outside the kept sets."""
    g = torch.Generator().manual_seed(seed)
    ids = b_cpu.draft_ids.clone()
    qi = b_cpu.q_indptr.tolist()
    V = b_cpu.spec.vocab
    for r in range(b_cpu.batch):
        if float(tau[r]) == 0.0:
            continue
        d0, k = qi[r] - r, qi[r + 1] - qi[r] - 1
        for i in range(k):
            if torch.rand((), generator=g) < 0.85:
                q, _, _ = oracle.filtered_row(b_cpu.draft_logits[d0 + i, :V], float(tau[r]), int(tk[r]), float(tp[r]))
                ids[d0 + i] = int(torch.multinomial(q, 1, generator=g))
    return dataclasses.replace(b_cpu, draft_ids=ids)


def _run(b_cpu, tau, tk, tp, **kw):
    b = b_cpu.to(DEV)
    acc, tok, ratio, ws = spx.rejection_sample(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample,
                                               temperature=None if tau is None else tau.to(DEV),
                                               top_k=None if tk is None else tk.to(DEV),
                                               top_p=None if tp is None else tp.to(DEV), **kw)
    torch.cuda.synchronize()
    return acc, tok, ratio, ws


def _report(name, rep):
    print(f"\n[{name}] exact {rep.exact}/{rep.requests}, accept-near-tie {rep.accept_near_tie}, cdf-near-tie {rep.cdf_near_tie}, "
          f"cdf-abs-near-tie {rep.cdf_abs_near_tie}, top-p-near-tie {rep.topp_near_tie}")


@pytest.mark.parametrize("idx,vocab", [(0, None), (1, 5000), (1, 128256), (4, 40000)])
def test_filtered_verification_matches_oracle(idx, vocab):
    spec = W.CONFIGS[idx] if idx == 0 else W.scaled(W.CONFIGS[idx], batch=16, ctx_div=64, vocab=vocab)
    b_cpu = W.generate(spec)
    tau, tk, tp = _params(b_cpu.batch, spec.vocab)
    b_cpu = _redraft(b_cpu, tau, tk, tp, seed=idx)
    acc, tok, _, ws = _run(b_cpu, tau, tk, tp)
    # top_k = 1 on rows whose target and draft agree on the maximum leaves a zero residual: reported, not an error
    assert int(ws.status.item()) & ~spx.DEV_DEGENERATE == 0
    rep = check_sampling(b_cpu, acc, tok, temperature=tau, top_k=tk, top_p=tp)
    _report(f"{spec.name} V={spec.vocab}", rep)
    assert not rep.hard_mismatch, rep
    assert rep.exact + rep.topp_near_tie >= rep.requests - 2


def test_filters_alone_and_off_switches():
    spec = W.scaled(W.CONFIGS[1], batch=12, ctx_div=64, vocab=20000)
    b_cpu = W.generate(spec)
    B = b_cpu.batch
    ones = torch.ones(B)
    # only top_k given, only top_p given, temperature absent
    for tk, tp in ((torch.full((B,), 40, dtype=torch.int32), None), (None, torch.full((B,), 0.8))):
        bb = _redraft(b_cpu, ones, tk if tk is not None else torch.zeros(B, dtype=torch.int32),
                      tp if tp is not None else ones, seed=3)
        acc, tok, _, ws = _run(bb, None, tk, tp)
        assert int(ws.status.item()) == 0
        rep = check_sampling(bb, acc, tok, top_k=tk, top_p=tp)
        assert not rep.hard_mismatch, rep
    # values that switch the filters off give the base rule's outputs
    b = b_cpu.to(DEV)
    acc0, tok0, _, _ = spx.rejection_sample(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample)
    acc1, tok1, _, ws = _run(b_cpu, None, torch.tensor([0, -1, spec.vocab, 10 ** 6] * 3, dtype=torch.int32), ones)
    assert int(ws.status.item()) == 0
    rep = check_sampling(b_cpu, acc1, tok1)
    assert not rep.hard_mismatch
    assert torch.equal(acc0, acc1) and torch.equal(tok0, tok1)


def test_top_k_one_equals_greedy_and_bad_top_p_is_reported():
    spec = W.scaled(W.CONFIGS[1], batch=8, ctx_div=64, vocab=30000)
    b_cpu = W.generate(spec)
    B = b_cpu.batch
    qi = b_cpu.q_indptr.tolist()
    # drafts = the target's argmax for most positions (harness side, torch.argmax)
    ids = b_cpu.draft_ids.clone()
    for r in range(B):
        for i in range(qi[r + 1] - qi[r] - 1):
            if (r + i) % 4:
                ids[qi[r] - r + i] = int(torch.argmax(b_cpu.target_logits[qi[r] + i, :spec.vocab].float()))
    b_cpu = dataclasses.replace(b_cpu, draft_ids=ids)
    tk1 = torch.ones(B, dtype=torch.int32)
    acc, tok, _, ws = _run(b_cpu, None, tk1, None)
    assert int(ws.status.item()) in (0, spx.DEV_DEGENERATE)
    ref = oracle.rejection_sample(b_cpu.target_logits, b_cpu.draft_logits, b_cpu.draft_ids, b_cpu.q_indptr, b_cpu.u_accept,
                                  b_cpu.u_sample, top_k=tk1)
    assert torch.equal(acc.cpu(), ref.accepted_len) and torch.equal(tok.cpu(), ref.out_tokens)
    # ... and, rows without ties for the maximum, equals greedy verification of the same drafts when the draft agrees
    tp = torch.full((B,), 0.9)
    tp[1], tp[4], tp[6] = 0.0, float("nan"), 1.5
    acc2, tok2, _, ws = _run(b_cpu, None, None, tp)
    assert int(ws.status.item()) & spx.DEV_BAD_PARAM
    for r in (1, 4, 6):
        assert int(acc2[r]) == 0 and bool((tok2[qi[r]:qi[r + 1]] == -1).all())
    good = torch.full((B,), 0.9)
    acc3, tok3, _, _ = _run(b_cpu, None, None, good)
    for r in (0, 2, 3, 5, 7):
        assert int(acc2[r]) == int(acc3[r]) and torch.equal(tok2[qi[r]:qi[r + 1]], tok3[qi[r]:qi[r + 1]])


def test_ties_at_the_thresholds():
    # coarse logits: many equal values, so the k-th value and the nucleus edge fall inside ties
    V, VS, B, k = 3000, 3000, 6, 2
    g = torch.Generator().manual_seed(5)
    T = torch.randint(-6, 7, (B * (k + 1), VS), generator=g).float().mul(0.5).to(torch.bfloat16)
    Dr = torch.randint(-6, 7, (B * k, VS), generator=g).float().mul(0.5).to(torch.bfloat16)
    qi = torch.arange(0, (B + 1) * (k + 1), k + 1, dtype=torch.int32)
    tk = torch.tensor([10, 300, 0, 0, 1, 2999], dtype=torch.int32)
    tp = torch.tensor([1.0, 1.0, 0.37, 0.9, 1.0, 0.5])
    ids = torch.zeros(B * k, dtype=torch.int32)
    for r in range(B):
        for i in range(k):
            q, _, _ = oracle.filtered_row(Dr[r * k + i], 1.0, int(tk[r]), float(tp[r]))
            ids[r * k + i] = int(torch.multinomial(q, 1, generator=g))
    ua, us = torch.rand(B * k, generator=g), torch.rand(B, generator=g)
    ref = oracle.rejection_sample(T, Dr, ids, qi, ua, us, top_k=tk, top_p=tp)
    acc, tok, _, ws = spx.rejection_sample(T.to(DEV), Dr.to(DEV), ids.to(DEV), qi.to(DEV), ua.to(DEV), us.to(DEV),
                                           top_k=tk.to(DEV), top_p=tp.to(DEV))
    torch.cuda.synchronize()

    class _B:
        pass
    bb = _B()
    bb.batch, bb.q_indptr, bb.u_accept, bb.u_sample = B, qi, ua, us
    bb.target_logits, bb.draft_logits, bb.draft_ids = T, Dr, ids
    bb.spec = type("S", (), {"vocab": V})
    rep = check_sampling(bb, acc, tok, ref, top_k=tk, top_p=tp)
    _report("ties", rep)
    assert not rep.hard_mismatch, (rep, acc.cpu().tolist(), ref.accepted_len.tolist())
    # every emitted token lies inside the oracle's kept set of its row
    for r in range(B):
        n = int(acc[r])
        y = int(tok[r * (k + 1) + n])
        p, _, _ = oracle.filtered_row(T[r * (k + 1) + n], 1.0, int(tk[r]), float(tp[r]))
        assert float(p[y]) > 0.0 or float(ref.margin[r]) < 1e-6


def test_crowded_threshold_bin():
    # tens of thousands of tokens share the value at which top-k / top-p cut (a block of equal logits, and a mass
    # of "masked" tokens far below the maximum): more than the kernel can park on chip, so it walks the row instead
    V, B, k = 60000, 4, 1
    g = torch.Generator().manual_seed(9)
    T = (torch.randn(B * (k + 1), V, generator=g) * 2).to(torch.bfloat16)
    Dr = (torch.randn(B * k, V, generator=g) * 2).to(torch.bfloat16)
    for rows in (T, Dr):
        rows[:, 5000:35000] = 1.0            # 30000 equal logits
        rows[:, 40000:] = -200.0             # 20000 masked tokens, all in the last distance bin
    qi = torch.arange(0, (B + 1) * (k + 1), k + 1, dtype=torch.int32)
    tk = torch.tensor([20000, 0, 45000, 50000], dtype=torch.int32)
    tp = torch.tensor([1.0, 0.6, 0.97, 1.0])
    ids = torch.zeros(B * k, dtype=torch.int32)
    for r in range(B):
        q, kept, _ = oracle.filtered_row(Dr[r], 1.0, int(tk[r]), float(tp[r]))
        ids[r] = int(torch.multinomial(q, 1, generator=g))
    assert oracle.filtered_row(T[0], 1.0, 20000, 1.0)[1] > 30000      # the whole tie is kept
    assert oracle.filtered_row(T[3 * 2], 1.0, 50000, 1.0)[1] == V     # cut inside the masked block: all of it kept
    ua, us = torch.rand(B * k, generator=g), torch.rand(B, generator=g)
    ref = oracle.rejection_sample(T, Dr, ids, qi, ua, us, top_k=tk, top_p=tp)
    acc, tok, _, ws = spx.rejection_sample(T.to(DEV), Dr.to(DEV), ids.to(DEV), qi.to(DEV), ua.to(DEV), us.to(DEV),
                                           top_k=tk.to(DEV), top_p=tp.to(DEV))
    torch.cuda.synchronize()

    class _B:
        pass
    bb = _B()
    bb.batch, bb.q_indptr, bb.u_accept, bb.u_sample = B, qi, ua, us
    bb.target_logits, bb.draft_logits, bb.draft_ids = T, Dr, ids
    bb.spec = type("S", (), {"vocab": V})
    rep = check_sampling(bb, acc, tok, ref, top_k=tk, top_p=tp)
    _report("crowded bin", rep)
    assert not rep.hard_mismatch, (rep, acc.cpu().tolist(), ref.accepted_len.tolist(), ref.margin.tolist())


@pytest.mark.parametrize("tie", [300, 4000, 20000])
def test_small_top_k_with_a_block_of_equal_logits_at_the_cut(tie):
    """A small K takes the short way: every logit at or above a lower bound of the K-th largest is a
    candidate, counted per exact value in a window of keys below the row maximum (bf16).  A block of
    equal logits at the cut - a few hundred, a few thousand, more than any list could hold - must
    not change the thresholds."""
    V, B, k = 60000, 4, 1                    # 30 sub-segments of 2048 tokens: K <= 30 qualifies
    g = torch.Generator().manual_seed(21 + tie)
    T = (torch.randn(B * (k + 1), V, generator=g)).to(torch.bfloat16)
    Dr = (torch.randn(B * k, V, generator=g)).to(torch.bfloat16)
    for rows in (T, Dr):
        rows[:, 1000:1000 + tie] = 6.0       # the tie: above every Gaussian logit, so it holds the cut for K > 10
        rows[:, 50000:50010] = 9.0           # ten equal logits above the tie
    qi = torch.arange(0, (B + 1) * (k + 1), k + 1, dtype=torch.int32)
    tk = torch.tensor([5, 11, 20, 30], dtype=torch.int32)
    tp = torch.tensor([1.0, 1.0, 0.9, 0.5])
    ids = torch.zeros(B * k, dtype=torch.int32)
    for r in range(B):
        q, kept, _ = oracle.filtered_row(Dr[r], 1.0, int(tk[r]), float(tp[r]))
        ids[r] = int(torch.multinomial(q, 1, generator=g))
    assert oracle.filtered_row(T[0], 1.0, 5, 1.0)[1] == 10             # cut inside the ten equal top logits: all kept
    assert oracle.filtered_row(T[2], 1.0, 11, 1.0)[1] == 10 + tie      # cut inside the tie: all of it kept
    ua, us = torch.rand(B * k, generator=g), torch.rand(B, generator=g)
    ref = oracle.rejection_sample(T, Dr, ids, qi, ua, us, top_k=tk, top_p=tp)
    acc, tok, _, ws = spx.rejection_sample(T.to(DEV), Dr.to(DEV), ids.to(DEV), qi.to(DEV), ua.to(DEV), us.to(DEV),
                                           top_k=tk.to(DEV), top_p=tp.to(DEV))
    torch.cuda.synchronize()
    assert int(ws.status.item()) in (0, spx.DEV_DEGENERATE)

    class _B:
        pass
    bb = _B()
    bb.batch, bb.q_indptr, bb.u_accept, bb.u_sample = B, qi, ua, us
    bb.target_logits, bb.draft_logits, bb.draft_ids = T, Dr, ids
    bb.spec = type("S", (), {"vocab": V})
    rep = check_sampling(bb, acc, tok, ref, top_k=tk, top_p=tp)
    assert not rep.hard_mismatch, rep
    assert rep.exact + rep.cdf_near_tie + rep.cdf_abs_near_tie + rep.accept_near_tie + rep.topp_near_tie == B


@pytest.mark.parametrize("masked", [float("-inf"), float(torch.finfo(torch.bfloat16).min), -3.0e4])
def test_masked_tokens_below_the_value_histogram(masked):
    """bf16 rows are settled by a histogram over the exact values that reaches a few ten thousand
    keys below the row maximum.  Masked tokens lie below it: they carry no mass, so cuts among the
    other tokens are still taken from the histogram; a top-k that reaches into the masked block, or a
    masked value that is still inside the histogram, must give the oracle's answer as well."""
    V, B, k = 40000, 6, 1
    g = torch.Generator().manual_seed(33)
    T = (torch.randn(B * (k + 1), V, generator=g) * 2.5).to(torch.bfloat16)
    Dr = (torch.randn(B * k, V, generator=g) * 2.5).to(torch.bfloat16)
    for rows in (T, Dr):
        rows[:, 28000:] = masked                 # 12000 masked tokens
        rows[:, 100:103] = 0.0                   # exact zeros of both signs
        rows[:, 103:105] = -0.0
        rows[:, 105] = 1e-30                     # values next to zero: thousands of keys from the other logits
        rows[:, 106] = -1e-30
    qi = torch.arange(0, (B + 1) * (k + 1), k + 1, dtype=torch.int32)
    tk = torch.tensor([0, 500, 35000, 0, 28000, 27999], dtype=torch.int32)   # 35000: the cut lies among the masked tokens
    tp = torch.tensor([0.9, 1.0, 1.0, 0.5, 0.999, 1.0])
    ids = torch.zeros(B * k, dtype=torch.int32)
    for r in range(B):
        q, kept, _ = oracle.filtered_row(Dr[r], 1.0, int(tk[r]), float(tp[r]))
        ids[r] = int(torch.multinomial(q, 1, generator=g))
    assert oracle.filtered_row(T[2 * 2], 1.0, 35000, 1.0)[1] == V
    ua, us = torch.rand(B * k, generator=g), torch.rand(B, generator=g)
    ref = oracle.rejection_sample(T, Dr, ids, qi, ua, us, top_k=tk, top_p=tp)
    acc, tok, _, ws = spx.rejection_sample(T.to(DEV), Dr.to(DEV), ids.to(DEV), qi.to(DEV), ua.to(DEV), us.to(DEV),
                                           top_k=tk.to(DEV), top_p=tp.to(DEV))
    torch.cuda.synchronize()
    assert int(ws.status.item()) in (0, spx.DEV_DEGENERATE)

    class _B:
        pass
    bb = _B()
    bb.batch, bb.q_indptr, bb.u_accept, bb.u_sample = B, qi, ua, us
    bb.target_logits, bb.draft_logits, bb.draft_ids = T, Dr, ids
    bb.spec = type("S", (), {"vocab": V})
    rep = check_sampling(bb, acc, tok, ref, top_k=tk, top_p=tp)
    _report(f"masked at {masked}", rep)
    assert not rep.hard_mismatch, (rep, acc.cpu().tolist(), ref.accepted_len.tolist(), ref.margin.tolist())
    assert rep.exact + rep.cdf_near_tie + rep.cdf_abs_near_tie + rep.accept_near_tie + rep.topp_near_tie == B


@pytest.mark.parametrize("V", [5003, 40001])
def test_ragged_vocabulary_and_unusual_rows(V):
    """A vocabulary that is no multiple of eight (the rows' padding holds poison the kernels must not
    read), and rows the named workloads do not have: all-negative logits, magnitudes next to zero, a
    wide spread, sharp and flat temperatures, coarse values with many ties, one dominant token."""
    B, k = 8, 2
    VS = (V + 7) // 8 * 8
    g = torch.Generator().manual_seed(77 + V)

    def rows(n):
        x = torch.randn(n, V, generator=g) * 2.5
        return x

    T, Dr = rows(B * (k + 1)), rows(B * k)
    for X, per in ((T, k + 1), (Dr, k)):
        X[1 * per:2 * per] = -20.0 + 5.0 * torch.randn(per, V, generator=g).clamp(-1.9, 1.9)     # all negative
        X[2 * per:3 * per] *= 1e-3                                                               # next to zero
        X[3 * per:4 * per] *= 3.2                                                                # wide
        X[6 * per:7 * per] = torch.randint(-4, 5, (per, V), generator=g).float()                 # ties
        X[7 * per:8 * per, 17] = 40.0                                                            # one dominant token
    T, Dr = T.to(torch.bfloat16), Dr.to(torch.bfloat16)
    Tp = torch.full((T.shape[0], VS), 1e4, dtype=torch.bfloat16)
    Dp = torch.full((Dr.shape[0], VS), 1e4, dtype=torch.bfloat16)
    Tp[:, :V], Dp[:, :V] = T, Dr
    qi = torch.arange(0, (B + 1) * (k + 1), k + 1, dtype=torch.int32)
    tk = torch.tensor([3, 0, 200, 0, 2, 1000, 0, 3], dtype=torch.int32)
    tp = torch.tensor([1.0, 0.9, 0.8, 0.3, 1.0, 0.95, 0.5, 0.9])
    tau = torch.tensor([1.0, 1.0, 1.0, 1.0, 0.05, 4.0, 1.0, 1.0])
    ids = torch.zeros(B * k, dtype=torch.int32)
    for r in range(B):
        for i in range(k):
            q, _, _ = oracle.filtered_row(Dr[r * k + i], float(tau[r]), int(tk[r]), float(tp[r]))
            ids[r * k + i] = int(torch.multinomial(q, 1, generator=g))
    ua, us = torch.rand(B * k, generator=g), torch.rand(B, generator=g)
    ref = oracle.rejection_sample(T, Dr, ids, qi, ua, us, temperature=tau, top_k=tk, top_p=tp)
    acc, tok, _, ws = spx.rejection_sample(Tp.to(DEV), Dp.to(DEV), ids.to(DEV), qi.to(DEV), ua.to(DEV), us.to(DEV), vocab=V,
                                           temperature=tau.to(DEV), top_k=tk.to(DEV), top_p=tp.to(DEV))
    torch.cuda.synchronize()
    assert int(ws.status.item()) in (0, spx.DEV_DEGENERATE)

    class _B:
        pass
    bb = _B()
    bb.batch, bb.q_indptr, bb.u_accept, bb.u_sample = B, qi, ua, us
    bb.target_logits, bb.draft_logits, bb.draft_ids = T, Dr, ids
    bb.spec = type("S", (), {"vocab": V})
    rep = check_sampling(bb, acc, tok, ref, temperature=tau, top_k=tk, top_p=tp)
    _report(f"ragged vocabulary {V}", rep)
    assert not rep.hard_mismatch, (rep, acc.cpu().tolist(), ref.accepted_len.tolist(), ref.margin.tolist())
    assert int(tok.max()) < V


@pytest.mark.parametrize("idx", [1, 2])
def test_full_size_filtered(idx):
    spec = W.CONFIGS[idx]
    b_cpu = W.generate(spec)
    tau, tk, tp = _params(b_cpu.batch, spec.vocab)
    b_cpu = _redraft(b_cpu, tau, tk, tp, seed=11)
    acc, tok, _, ws = _run(b_cpu, tau, tk, tp)
    assert int(ws.status.item()) & ~spx.DEV_DEGENERATE == 0
    rep = check_sampling(b_cpu, acc, tok, temperature=tau, top_k=tk, top_p=tp)
    _report(f"{spec.name}, mixed filters", rep)
    assert not rep.hard_mismatch, rep
    # repeated launches agree bit for bit (integer atomics: no dependence on the order of arrival)
    for _ in range(2):
        acc2, tok2, _, _ = _run(b_cpu, tau, tk, tp)
        assert torch.equal(acc, acc2) and torch.equal(tok, tok2)
