"""Seeded synthetic inputs for the speculative-decoding verify step.

This module only *draws inputs*: shapes, lengths, page tables, Gaussian tensors, uniforms and
draft token ids.  It contains none of the verify step's arithmetic (no attention, no softmax,
no accept test) and is the one module that both the CPU oracle's tests and the CUDA path's
tests/benchmark use, so that both sides see the same bits.

The five named workloads stand in for the serving workloads of the paper's evaluation
(Section 7: Llama-3 / Qwen-3 models on public chat benchmarks, fixed batch 64 in Table 3),
whose datasets and weights are not available: the *shapes* are those of the named model
families and the draft noise is chosen so that acceptance rates fall in the range the paper's
Table 4 reports.

Recipe common to all workloads (seed = 20260934 + workload index):
  * Q, K, V ~ N(0,1), cast to the KV dtype; the pools are ``[num_pages, Hkv, P, D]`` ("HND")
    or ``[num_pages, P, Hkv, D]`` ("NHD"), K and V separate;
  * target logits ~ N(0, sigma_t^2); draft logits = target + N(0, sigma_d^2), both cast to the
    logits dtype after the add;
  * draft token i is drawn from the distribution the stored draft row i defines, by the
    Gumbel-max trick (argmax of logits + Gumbel noise) so that no softmax is evaluated here;
  * u_accept, u_sample are uniform on the 2^-24 grid in [0,1);
  * context lengths count the k+1 new positions; block tables are random page permutations
    (the "fragmented" workload draws its pages from a pool twice as large, leaving holes);
  * slots that must never be read (tail of each last page, unused pages) hold a large finite
    poison value, and unused block-table entries are -1.
Lengths, draft counts and page tables are always drawn with a CPU generator, so they do not
depend on the device the tensors are created on.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import torch

POISON = 1.0e4
BASE_SEED = 20260934


@dataclass(frozen=True)
class WorkloadSpec:
    name: str
    index: int
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    vocab: int
    dtype: str                      # "bf16" or "fp32": Q/K/V/O and logits
    ctx: Tuple                      # ("uniform", lo, hi) | ("lognormal", median, sigma, lo, cap) | ("const", L)
    k: Tuple                        # ("const", k) | ("choice", (k0, k1, ...))
    sigma_t: float = 3.0
    sigma_d: float = 1.0
    pool_factor: int = 1            # 2 = fragmented pool (half of the pages unused)

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32


CONFIGS: List[WorkloadSpec] = [
    WorkloadSpec("tiny-fp32", 0, 4, 8, 2, 64, 16, 1024, "fp32", ("uniform", 32, 256), ("const", 4)),
    WorkloadSpec("llama3-8b", 1, 64, 32, 8, 128, 16, 128256, "bf16", ("uniform", 512, 4096), ("const", 5)),
    WorkloadSpec("llama3-70b", 2, 128, 64, 8, 128, 16, 128256, "bf16",
                 ("lognormal", 1024, 1.0, 16, 8192), ("const", 3), sigma_d=0.5),
    WorkloadSpec("long-context", 3, 16, 32, 8, 128, 32, 32000, "bf16", ("const", 32768), ("const", 8),
                 sigma_d=2.0),
    WorkloadSpec("selective-mix", 4, 256, 32, 8, 128, 16, 128256, "bf16", ("uniform", 128, 8192),
                 ("choice", (0, 2, 4, 6)), pool_factor=2),
]


def scaled(spec: WorkloadSpec, batch: Optional[int] = None, ctx_div: int = 1,
           vocab: Optional[int] = None, name_suffix: str = "-small") -> WorkloadSpec:
    """A reduced copy of a workload: fewer requests, contexts divided by ``ctx_div``, smaller vocab."""
    ctx = spec.ctx
    kmax = max(spec.k[1]) if spec.k[0] == "choice" else spec.k[1]
    floor = kmax + 1
    if ctx_div > 1:
        if ctx[0] == "uniform":
            ctx = ("uniform", max(floor, ctx[1] // ctx_div), max(floor, ctx[2] // ctx_div))
        elif ctx[0] == "lognormal":
            ctx = ("lognormal", max(floor, ctx[1] // ctx_div), ctx[2], max(floor, ctx[3] // ctx_div),
                   max(floor, ctx[4] // ctx_div))
        else:
            ctx = ("const", max(floor, ctx[1] // ctx_div))
    return dataclasses.replace(spec, name=spec.name + name_suffix, batch=batch or spec.batch, ctx=ctx,
                               vocab=vocab or spec.vocab)


@dataclass
class VerifyBatch:
    spec: WorkloadSpec
    layout: str
    num_pages: int
    q: torch.Tensor                 # [TQ, Hq, D]
    k_cache: torch.Tensor           # pool
    v_cache: torch.Tensor           # pool
    kv_strides: Tuple[int, int, int]  # (page, head, token) element strides
    block_table: torch.Tensor       # [B, max_pages] int32, -1 = unused
    seq_lens: torch.Tensor          # [B] int32
    q_indptr: torch.Tensor          # [B+1] int32
    target_logits: torch.Tensor     # [TQ, V]
    draft_logits: torch.Tensor      # [TD, V]
    draft_ids: torch.Tensor         # [TD] int32
    u_accept: torch.Tensor          # [TD] fp32
    u_sample: torch.Tensor          # [B] fp32
    seq_lens_host: List[int] = field(default_factory=list)
    k_host: List[int] = field(default_factory=list)

    _TENSORS = ("q", "k_cache", "v_cache", "block_table", "seq_lens", "q_indptr", "target_logits",
                "draft_logits", "draft_ids", "u_accept", "u_sample")

    def to(self, device) -> "VerifyBatch":
        kw = {n: getattr(self, n).to(device) for n in self._TENSORS}
        return dataclasses.replace(self, **kw)

    def clone(self) -> "VerifyBatch":
        kw = {n: getattr(self, n).clone() for n in self._TENSORS}
        return dataclasses.replace(self, **kw)

    @property
    def batch(self) -> int:
        return len(self.seq_lens_host)

    @property
    def total_q(self) -> int:
        return sum(self.k_host) + len(self.k_host)

    @property
    def total_d(self) -> int:
        return sum(self.k_host)

    def kv_bytes(self) -> int:
        """Bytes of K and V the step must read: exact tokens, not page-rounded."""
        s = self.spec
        return sum(self.seq_lens_host) * s.num_kv_heads * s.head_dim * 2 * self.q.element_size()

    def logits_bytes(self) -> int:
        """Nominal logits bytes: every target and draft row once."""
        return (self.total_q + self.total_d) * self.spec.vocab * self.target_logits.element_size()

    def host_copy_bytes(self) -> int:
        return sum(getattr(self, n).numel() * getattr(self, n).element_size() for n in self._TENSORS)


def _draw_lengths(spec: WorkloadSpec, g: torch.Generator) -> Tuple[List[int], List[int]]:
    B = spec.batch
    if spec.k[0] == "const":
        ks = [int(spec.k[1])] * B
    else:
        choices = torch.tensor(spec.k[1])
        ks = choices[torch.randint(0, len(choices), (B,), generator=g)].tolist()
    c = spec.ctx
    if c[0] == "uniform":
        Ls = torch.randint(c[1], c[2] + 1, (B,), generator=g).tolist()
    elif c[0] == "lognormal":
        z = torch.randn(B, generator=g, dtype=torch.float64)
        Ls = torch.floor(torch.exp(math.log(c[1]) + c[2] * z)).clamp(c[3], c[4]).to(torch.int64).tolist()
    else:
        Ls = [int(c[1])] * B
    Ls = [max(int(L), k + 1) for L, k in zip(Ls, ks)]
    return Ls, [int(k) for k in ks]


def _uniform24(n: int, g: torch.Generator, device) -> torch.Tensor:
    ints = torch.randint(0, 1 << 24, (n,), generator=g, device=device, dtype=torch.int32)
    return ints.to(torch.float32) / float(1 << 24)


def generate(spec: WorkloadSpec, device="cpu", layout: str = "HND", seed: Optional[int] = None,
             extra_table_cols: int = 2) -> VerifyBatch:
    """Draw one batch of the workload on ``device`` (tensors) with CPU-drawn shapes."""
    seed = spec.seed if seed is None else seed
    device = torch.device(device)
    g_cpu = torch.Generator(device="cpu")
    g_cpu.manual_seed(seed)
    g = torch.Generator(device=device)
    g.manual_seed(seed + 1)
    dt = spec.torch_dtype
    B, Hq, Hkv, D, P, V = (spec.batch, spec.num_q_heads, spec.num_kv_heads, spec.head_dim,
                           spec.page_size, spec.vocab)

    Ls, ks = _draw_lengths(spec, g_cpu)
    pages_per_req = [(L + P - 1) // P for L in Ls]
    used_pages = sum(pages_per_req)
    num_pages = used_pages * spec.pool_factor
    perm = torch.randperm(num_pages, generator=g_cpu)[:used_pages].to(torch.int32)
    max_pages = max(pages_per_req) + extra_table_cols
    block_table = torch.full((B, max_pages), -1, dtype=torch.int32)
    off = 0
    for r, n in enumerate(pages_per_req):
        block_table[r, :n] = perm[off:off + n]
        off += n

    q_indptr = [0]
    for k in ks:
        q_indptr.append(q_indptr[-1] + k + 1)
    TQ = q_indptr[-1]
    TD = TQ - B

    # KV pools
    if layout == "HND":
        shape = (num_pages, Hkv, P, D)
        strides = (Hkv * P * D, P * D, D)
    elif layout == "NHD":
        shape = (num_pages, P, Hkv, D)
        strides = (P * Hkv * D, D, Hkv * D)
    else:
        raise ValueError(layout)
    k_cache = torch.empty(shape, dtype=dt, device=device).normal_(generator=g)
    v_cache = torch.empty(shape, dtype=dt, device=device).normal_(generator=g)
    # poison what must never be read
    if spec.pool_factor > 1:
        mask = torch.ones(num_pages, dtype=torch.bool)
        mask[perm.long()] = False
        unused = mask.nonzero().flatten().to(device)
        k_cache[unused] = POISON
        v_cache[unused] = -POISON
    for r, L in enumerate(Ls):
        tail = L % P
        if tail:
            page = int(block_table[r, pages_per_req[r] - 1])
            if layout == "HND":
                k_cache[page, :, tail:, :] = POISON
                v_cache[page, :, tail:, :] = -POISON
            else:
                k_cache[page, tail:, :, :] = POISON
                v_cache[page, tail:, :, :] = -POISON

    q = torch.empty((TQ, Hq, D), dtype=dt, device=device).normal_(generator=g)

    # logits: draft = target + noise, cast after the add
    t32 = torch.empty((TQ, V), dtype=torch.float32, device=device).normal_(generator=g) * spec.sigma_t
    target_logits = t32.to(dt)
    if TD > 0:
        # target rows that have a draft partner: positions 0..k_r-1 of each request
        rows = torch.tensor([q_indptr[r] + i for r in range(B) for i in range(ks[r])],
                            dtype=torch.long, device=device)
        d32 = t32[rows] + torch.empty((TD, V), dtype=torch.float32, device=device).normal_(generator=g) * spec.sigma_d
        draft_logits = d32.to(dt)
        del d32
        # Gumbel-max draw from the distribution the stored draft row defines
        u = torch.empty((TD, V), dtype=torch.float32, device=device).uniform_(generator=g)
        u = u.clamp_(min=1e-30, max=1.0 - 2.0 ** -24)
        gumbel = -torch.log(-torch.log(u))
        draft_ids = torch.argmax(draft_logits.to(torch.float32) + gumbel, dim=1).to(torch.int32)
        del u, gumbel
    else:
        draft_logits = torch.empty((0, V), dtype=dt, device=device)
        draft_ids = torch.empty((0,), dtype=torch.int32, device=device)
    del t32

    return VerifyBatch(
        spec=spec, layout=layout, num_pages=num_pages, q=q, k_cache=k_cache, v_cache=v_cache,
        kv_strides=strides, block_table=block_table.to(device),
        seq_lens=torch.tensor(Ls, dtype=torch.int32, device=device),
        q_indptr=torch.tensor(q_indptr, dtype=torch.int32, device=device),
        target_logits=target_logits, draft_logits=draft_logits, draft_ids=draft_ids,
        u_accept=_uniform24(TD, g, device), u_sample=_uniform24(B, g, device),
        seq_lens_host=Ls, k_host=ks)
