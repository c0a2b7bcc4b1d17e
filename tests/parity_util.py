"""Helpers shared by the GPU parity tests: run both sides on one batch and compare.

Tolerances (stated where they are used as well):
  * attention, bf16: max abs error <= 2e-2 (contract) and, because that bound is loose next to
    the signal at long context, also relative RMS error <= 1e-2 and |LSE error| <= 2e-3;
    fp32: max abs <= 1e-4, relative RMS <= 1e-5, |LSE error| <= 1e-4.
  * sampling: accepted lengths and token ids bit-exact, except requests in which some consulted
    draft has |p/q - u| < 1e-6 (accept-class near tie) or whose target s*R lies within 1e-6*R of
    the CDF interval of the token the GPU chose (cdf-class near tie, an fp32 scan cannot
    reproduce a float64 sequential cumulative sum bit for bit).  Both classes are counted.
  * sampling at a temperature other than 1: the same, plus a third counted class.  At low
    temperature p and q can both be within fp32 resolution of the same one-hot row, so the residual
    max(0, p - q) is a difference of nearly equal fp32 numbers and its total mass R can fall below
    what fp32 probabilities resolve at all (R ~ 1e-9 occurs at tau = 0.05).  A band relative to R is
    then meaningless for an fp32 kernel; the class is stated in absolute probability mass instead:
    the GPU's token is tolerated iff s*R lies within 2^-22 (four fp32 ulps of unit mass, the
    resolution of p and q near 1) of the oracle's cumulative interval of that token.
  * top-p filtering: the kept set is decided by comparing a running mass with top_p; the kernel
    sums fp32 exponentials (exactly, in fixed point), the oracle float64 ones.  A request in which
    some consulted row's crossing came within 1e-6 (in units of the survivors' mass) of tipping to
    the neighbouring value is exempt as a whole, and counted.  top-k is exact (stored values).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import torch

import oracle
import paper_2609_34370_b200 as spx

ATTN_TOL = {
    torch.bfloat16: dict(max_abs=2e-2, rel_rms=1e-2, lse_abs=2e-3),
    torch.float32: dict(max_abs=1e-4, rel_rms=1e-5, lse_abs=1e-4),
}
ACCEPT_BAND = 1e-6
CDF_BAND = 1e-6
CDF_ABS_BAND = 2.0 ** -22       # variants only: absolute probability mass
TOPP_BAND = 1e-6                # top-p only: margin of the crossing, in units of the survivors' mass


def gpu_attention(b, ws=None, **kw):
    s = b.spec
    out, lse, ws = spx.verify_attention(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens,
                                        b.q_indptr, s.num_kv_heads, s.page_size, b.num_pages, ws=ws, **kw)
    torch.cuda.synchronize()
    return out, lse, ws


def oracle_attention(b_cpu, req_list=None):
    s = b_cpu.spec
    return oracle.verify_attention(b_cpu.q, b_cpu.k_cache, b_cpu.v_cache, b_cpu.kv_strides, b_cpu.block_table,
                                   b_cpu.seq_lens, b_cpu.q_indptr, s.num_kv_heads, s.page_size, b_cpu.num_pages,
                                   req_list=req_list)


def rows_of(b, reqs):
    rows = []
    qi = b.q_indptr.tolist()
    for r in reqs:
        rows.extend(range(qi[r], qi[r + 1]))
    return torch.tensor(rows, dtype=torch.long)


def check_attention(b, out_gpu, lse_gpu, out_ref, lse_ref, reqs=None):
    """Compare GPU output with the oracle's on the rows of `reqs` (all requests if None)."""
    tol = ATTN_TOL[b.q.dtype]
    rows = rows_of(b, reqs if reqs is not None else range(b.batch))
    og = out_gpu.detach().cpu().double()[rows]
    lg = lse_gpu.detach().cpu().double()[rows]
    orf, lrf = out_ref[rows], lse_ref[rows]
    assert torch.isfinite(og).all() and torch.isfinite(lg).all()
    max_abs = float((og - orf).abs().max())
    rel_rms = float((og - orf).norm() / orf.norm())
    lse_abs = float((lg - lrf).abs().max())
    stats = dict(max_abs=max_abs, rel_rms=rel_rms, lse_abs=lse_abs)
    assert max_abs <= tol["max_abs"], stats
    assert rel_rms <= tol["rel_rms"], stats
    assert lse_abs <= tol["lse_abs"], stats
    return stats


@dataclass
class SampleReport:
    requests: int = 0
    exact: int = 0
    accept_near_tie: int = 0
    cdf_near_tie: int = 0
    cdf_abs_near_tie: int = 0           # requests at a temperature other than 1 only
    topp_near_tie: int = 0              # requests whose top-p crossing was within TOPP_BAND of tipping
    hard_mismatch: List[int] = field(default_factory=list)
    accept_band_eligible: int = 0       # consulted drafts inside the accept band (oracle side)


def check_sampling(b_cpu, acc_gpu, tok_gpu, ref: Optional[oracle.SampleResult] = None,
                   temperature: Optional[torch.Tensor] = None, top_k: Optional[torch.Tensor] = None,
                   top_p: Optional[torch.Tensor] = None) -> SampleReport:
    """Bit-exactness of (accepted_len, out_tokens) outside the two counted near-tie classes.
    Greedy requests (temperature 0) have no near-tie class: they must match exactly."""
    if ref is None:
        ref = oracle.rejection_sample(b_cpu.target_logits, b_cpu.draft_logits, b_cpu.draft_ids, b_cpu.q_indptr,
                                      b_cpu.u_accept, b_cpu.u_sample, temperature=temperature, top_k=top_k, top_p=top_p)
    acc_gpu = acc_gpu.detach().cpu()
    tok_gpu = tok_gpu.detach().cpu()
    qi = b_cpu.q_indptr.tolist()
    rep = SampleReport(requests=b_cpu.batch)
    rho = ref.rho
    ua = b_cpu.u_accept.double()
    near = (rho - ua).abs() < ACCEPT_BAND
    rep.accept_band_eligible = int(near.sum())
    for r in range(b_cpu.batch):
        t0, t1 = qi[r], qi[r + 1]
        d0, k = t0 - r, t1 - t0 - 1
        n_o, n_g = int(ref.accepted_len[r]), int(acc_gpu[r])
        if n_o == n_g and torch.equal(ref.out_tokens[t0:t1], tok_gpu[t0:t1]):
            rep.exact += 1
            continue
        tau = 1.0 if temperature is None else float(temperature[r])
        if not tau > 0.0:
            rep.hard_mismatch.append(r)
            continue
        if ref.margin is not None and float(ref.margin[r]) < TOPP_BAND:
            rep.topp_near_tie += 1
            continue
        tk = 0 if top_k is None else int(top_k[r])
        tp = 1.0 if top_p is None else float(top_p[r])
        upto = min(max(n_o, n_g), k - 1)
        if k > 0 and bool(near[d0:d0 + upto + 1].any()):
            rep.accept_near_tie += 1
            continue
        if n_o == n_g and torch.equal(ref.out_tokens[t0:t0 + n_o], tok_gpu[t0:t0 + n_o]) and \
                bool((tok_gpu[t0 + n_o + 1:t1] == -1).all()):
            y_g = int(tok_gpu[t0 + n_o])
            if 0 <= y_g < b_cpu.spec.vocab:
                cdf, R = oracle.emit_cdf(r, n_o, b_cpu.target_logits, b_cpu.draft_logits, b_cpu.q_indptr, tau=tau,
                                         top_k=tk, top_p=tp)
                target = float(b_cpu.u_sample[r]) * R
                lo = float(cdf[y_g - 1]) if y_g > 0 else 0.0
                hi = float(cdf[y_g])
                if hi > lo and lo - CDF_BAND * R <= target <= hi + CDF_BAND * R:
                    rep.cdf_near_tie += 1
                    continue
                if (tau != 1.0 or tk > 0 or tp < 1.0) and lo - CDF_ABS_BAND <= target <= hi + CDF_ABS_BAND:
                    rep.cdf_abs_near_tie += 1
                    continue
        rep.hard_mismatch.append(r)
    return rep


def gpu_sample(b, **kw):
    acc, tok, ratio, ws = spx.rejection_sample(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr,
                                               b.u_accept, b.u_sample, **kw)
    torch.cuda.synchronize()
    return acc, tok, ratio, ws
