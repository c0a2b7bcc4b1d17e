"""Helpers shared by the GPU parity tests: run both sides on one batch and compare.

Tolerances (stated where they are used as well):
  * attention, bf16: max abs error <= 2e-2 (contract) and, because that bound is loose next to
    the signal at long context, also relative RMS error <= 1e-2 and |LSE error| <= 2e-5;
    fp32: max abs <= 1e-4, relative RMS <= 1e-5, |LSE error| <= 2e-5.
    The LSE gate is the one that sees a lost page: leaving 16 of L tokens out of a softmax over
    N(0,1) scores lowers LSE by about 16/L, i.e. 4e-3 at L = 4096 and 5e-4 at L = 32768, while the
    output moves by only 3e-3 and 4e-4.  The kernels form the row sums in fp32 from exact bf16
    products; observed |LSE error| on the five workloads at full size is 1.2e-6 to 1.4e-6, so the
    gate sits 15x above the arithmetic's noise and 20x below the smallest lost-page signal.  (LSE
    comes back as fp32, so four units in the last place of the value are allowed on top.)
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
    torch.bfloat16: dict(max_abs=2e-2, rel_rms=1e-2, lse_abs=2e-5),
    torch.float32: dict(max_abs=1e-4, rel_rms=1e-5, lse_abs=2e-5),
}
ACCEPT_BAND = 1e-6
CDF_BAND = 1e-6
CDF_ABS_BAND = 2.0 ** -22       # variants only: absolute probability mass
TOPP_BAND = 1e-6                # top-p only: margin of the crossing, in units of the survivors' mass


GUARD_BYTES = 4096              # guard band on each side of every buffer the library writes
GUARD_BYTE = 0xC3


class Guarded:
    """A device buffer with a guard band before and after it.  The bands are filled with a fixed byte
    and must read back unchanged after the call: the stand-in for a memory checker on the buffers the
    library writes (workspace, attention output, LSE, accepted lengths, tokens)."""

    def __init__(self, shape, dtype, device, name):
        self.name = name
        nbytes = int(torch.tensor([], dtype=dtype).element_size())
        for d in (shape if isinstance(shape, (tuple, list, torch.Size)) else (shape,)):
            nbytes *= int(d)
        self.nbytes = nbytes
        pad = (-nbytes) % 256                                       # the back band starts on a 256-byte boundary
        self.raw = torch.full((GUARD_BYTES + nbytes + pad + GUARD_BYTES,), GUARD_BYTE, dtype=torch.uint8, device=device)
        self.view = self.raw[GUARD_BYTES:GUARD_BYTES + nbytes].view(dtype).view(shape)
        assert self.raw.device.type != "cuda" or self.view.data_ptr() % 256 == 0   # the library wants 256-byte aligned scratch

    def check(self):
        front = self.raw[:GUARD_BYTES]
        back = self.raw[GUARD_BYTES + self.nbytes:]
        assert bool((front == GUARD_BYTE).all()), f"write before the start of {self.name}"
        assert bool((back == GUARD_BYTE).all()), f"write past the end of {self.name}"


def guarded_workspace(nbytes, device, name="workspace"):
    g = Guarded((nbytes,), torch.uint8, device, name)
    return g, spx.Workspace(g.view, torch.zeros(1, dtype=torch.int32, device=device))


def gpu_attention(b, ws=None, **kw):
    """spx_verify_attention with the output, the LSE and (unless the caller brings one) the workspace
    inside guard bands, which are checked after the call."""
    from paper_2609_34370_b200 import binding
    s = b.spec
    dev = b.q.device
    g_out = Guarded(tuple(b.q.shape), b.q.dtype, dev, "attention output")
    g_lse = Guarded(tuple(b.q.shape[:2]), torch.float32, dev, "lse")
    guards = [g_out, g_lse]
    if ws is None:
        a = binding.make_attn_args(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                                   s.num_kv_heads, s.page_size, b.num_pages, g_out.view, g_lse.view,
                                   kw.get("sm_scale", 0.0), kw.get("max_q_len", 0))
        g_ws, ws = guarded_workspace(spx.workspace_size(a, None), dev, "attention workspace")
        ws._guard = g_ws
    if getattr(ws, "_guard", None) is not None:
        guards.append(ws._guard)
    out, lse, ws = spx.verify_attention(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens,
                                        b.q_indptr, s.num_kv_heads, s.page_size, b.num_pages, out=g_out.view,
                                        lse=g_lse.view, ws=ws, **kw)
    torch.cuda.synchronize()
    for g in guards:
        g.check()
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
    # LSE is returned as fp32: beside the absolute gate, four units in the last place of the value
    # itself (a needle key puts LSE near 60, where one fp32 step is 4e-6)
    lse_abs = float(((lg - lrf).abs() - lrf.abs() * 2.0 ** -21).clamp(min=0).max())
    stats = dict(max_abs=max_abs, rel_rms=rel_rms, lse_abs=lse_abs, rows=int(rows.numel()))
    print(f"\n[attention parity {getattr(b.spec, 'name', '?')}] " + ", ".join(
        f"{k} {v:.3e}" if isinstance(v, float) else f"{k} {v}" for k, v in stats.items()))
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
    """spx_rejection_sample with accepted lengths, tokens and workspace inside checked guard bands."""
    from paper_2609_34370_b200 import binding
    dev = b.target_logits.device
    B, TQ = b.q_indptr.numel() - 1, b.target_logits.shape[0]
    g_acc = Guarded((B,), torch.int32, dev, "accepted_len")
    g_tok = Guarded((TQ,), torch.int32, dev, "out_tokens")
    guards = [g_acc, g_tok]
    ws = kw.pop("ws", None)
    if ws is None:
        sa = binding.make_sample_args(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample,
                                      g_acc.view, g_tok.view, None, kw.get("vocab"), kw.get("temperature"),
                                      kw.get("top_k"), kw.get("top_p"), kw.get("target_tile_stats"))
        g_ws, ws = guarded_workspace(spx.workspace_size(None, sa), dev, "sampling workspace")
        ws._guard = g_ws
    if getattr(ws, "_guard", None) is not None:
        guards.append(ws._guard)
    acc, tok, ratio, ws = spx.rejection_sample(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr,
                                               b.u_accept, b.u_sample, ws=ws, accepted=g_acc.view, tokens=g_tok.view,
                                               **kw)
    torch.cuda.synchronize()
    for g in guards:
        g.check()
    return acc, tok, ratio, ws
