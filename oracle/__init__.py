"""CPU oracle for the speculative-decoding verify step.  TEST INFRASTRUCTURE ONLY.

A thin ctypes wrapper around ``spx_oracle.c`` (plain C, float64 arithmetic, OpenMP over
independent items).  Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA library and its Python binding never do, and the two share no
code.  See the header of ``spx_oracle.c`` for what each function follows and how it is pinned.

All tensors are CPU ``torch`` tensors (bf16 or fp32 for data, int32 for indices); outputs are
float64 / int32 CPU tensors.
"""
from __future__ import annotations

import ctypes
import ctypes as c
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spx_oracle.c")
_LIB_PATH = os.path.join(_HERE, "libspx_oracle.so")

BF16, F32 = 0, 1
OK, ERR_ARG, ERR_LEN, ERR_PAGE, ERR_TOKEN, ERR_ALLOC, ERR_PARAM = 0, 1, 2, 3, 4, 5, 6
FLAG_DEGENERATE = 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP).  Returns the library path."""
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-o", _LIB_PATH,
               _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB_PATH)
        c = ctypes
        lib.oracle_num_threads.restype = c.c_int
        lib.oracle_verify_attention.restype = c.c_int
        lib.oracle_verify_attention.argtypes = [
            c.c_int32, c.c_int32, c.c_int32, c.c_int32, c.c_int32, c.c_int64, c.c_int32, c.c_int32,
            c.c_double, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int64, c.c_int64, c.c_int64,
            c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int32, c.c_void_p, c.c_void_p]
        lib.oracle_softmax_row.restype = None
        lib.oracle_softmax_row.argtypes = [c.c_void_p, c.c_int32, c.c_int64, c.c_int64, c.c_void_p]
        lib.oracle_residual.restype = c.c_double
        lib.oracle_residual.argtypes = [c.c_void_p, c.c_void_p, c.c_int64, c.c_void_p]
        lib.oracle_inverse_cdf.restype = c.c_int64
        lib.oracle_inverse_cdf.argtypes = [c.c_void_p, c.c_int64, c.c_double, c.c_double,
                                           c.c_void_p, c.c_void_p]
        lib.oracle_rejection_sample.restype = c.c_int
        lib.oracle_rejection_sample.argtypes = [
            c.c_int32, c.c_int64, c.c_int64, c.c_int32, c.c_void_p, c.c_void_p, c.c_void_p,
            c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
            c.c_void_p, c.c_void_p, c.c_void_p]
        lib.oracle_emit_cdf.restype = c.c_double
        lib.oracle_emit_cdf.argtypes = [c.c_int32, c.c_int32, c.c_int64, c.c_int64, c.c_int32,
                                        c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
        lib.oracle_kv_append.restype = c.c_int
        lib.oracle_kv_append.argtypes = [c.c_int32, c.c_int32, c.c_int32, c.c_int32, c.c_int64, c.c_int32, c.c_int32,
                                         c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int64, c.c_int64, c.c_int64,
                                         c.c_void_p, c.c_void_p, c.c_void_p]
        lib.oracle_kv_rollback.restype = c.c_int
        lib.oracle_kv_rollback.argtypes = [c.c_int32, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"oracle accepts bf16 or fp32 data, got {t.dtype}")


def _cpu(t: torch.Tensor, dtype=None) -> torch.Tensor:
    assert t.device.type == "cpu", "oracle inputs must be host tensors"
    if dtype is not None:
        assert t.dtype == dtype, (t.dtype, dtype)
    return t


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle returned error code {code}")
        self.code = code


def verify_attention(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
                     kv_strides: Sequence[int], block_table: torch.Tensor, seq_lens: torch.Tensor,
                     q_indptr: torch.Tensor, num_kv_heads: int, page_size: int, num_pages: int,
                     sm_scale: float = 0.0, req_list: Optional[Sequence[int]] = None):
    """Attention of every request's k+1 query rows over its paged cache, in float64.

    ``q`` is [TQ, Hq, D]; ``k_cache``/``v_cache`` are pools addressed by
    ``kv_strides = (page, head, token)`` element strides with D contiguous.  Returns
    ``(out [TQ,Hq,D] float64, lse [TQ,Hq] float64)``; with ``req_list`` only those requests'
    rows are computed (the rest stay NaN).
    """
    lib = _load()
    q = _cpu(q).contiguous()
    dt = _dtype_code(q)
    assert _dtype_code(k_cache) == dt and _dtype_code(v_cache) == dt
    TQ, Hq, D = q.shape
    B = seq_lens.numel()
    bt = _cpu(block_table, torch.int32).contiguous()
    sl = _cpu(seq_lens, torch.int32).contiguous()
    qi = _cpu(q_indptr, torch.int32).contiguous()
    out = torch.full((TQ, Hq, D), float("nan"), dtype=torch.float64)
    lse = torch.full((TQ, Hq), float("nan"), dtype=torch.float64)
    rl = None
    n_rl = 0
    if req_list is not None:
        rl = torch.tensor(list(req_list), dtype=torch.int32)
        n_rl = rl.numel()
    st = lib.oracle_verify_attention(
        B, Hq, num_kv_heads, D, page_size, num_pages, bt.shape[1] if bt.dim() == 2 else 0, dt,
        float(sm_scale), _ptr(q), _ptr(k_cache), _ptr(v_cache), int(kv_strides[0]),
        int(kv_strides[1]), int(kv_strides[2]), _ptr(bt), _ptr(sl), _ptr(qi), _ptr(rl), n_rl,
        _ptr(out), _ptr(lse))
    if st != OK:
        raise OracleError(st)
    return out, lse


def softmax_row(logits_row: torch.Tensor, tau: Optional[float] = None) -> torch.Tensor:
    """Step 1 of the sampling rule: float64 softmax of one stored logits row (at temperature tau)."""
    lib = _load()
    row = _cpu(logits_row).contiguous()
    p = torch.empty(row.numel(), dtype=torch.float64)
    if tau is None:
        lib.oracle_softmax_row(_ptr(row), _dtype_code(row), 0, row.numel(), _ptr(p))
    else:
        lib.oracle_softmax_row_tau.restype = None
        lib.oracle_softmax_row_tau.argtypes = [c.c_void_p, c.c_int32, c.c_int64, c.c_int64, c.c_double, c.c_void_p]
        lib.oracle_softmax_row_tau(_ptr(row), _dtype_code(row), 0, row.numel(), float(tau), _ptr(p))
    return p


def argmax_row(logits_row: torch.Tensor) -> int:
    """Greedy choice of one stored logits row: the lowest id attaining the maximum."""
    lib = _load()
    row = _cpu(logits_row).contiguous()
    lib.oracle_argmax_row.restype = c.c_int64
    lib.oracle_argmax_row.argtypes = [c.c_void_p, c.c_int32, c.c_int64, c.c_int64]
    return int(lib.oracle_argmax_row(_ptr(row), _dtype_code(row), 0, row.numel()))


def residual(p: torch.Tensor, q: torch.Tensor):
    """Step 3: r = max(0, p - q) and its mass R."""
    lib = _load()
    p = _cpu(p, torch.float64).contiguous()
    q = _cpu(q, torch.float64).contiguous()
    r = torch.empty_like(p)
    R = lib.oracle_residual(_ptr(p), _ptr(q), p.numel(), _ptr(r))
    return r, float(R)


def inverse_cdf(r: torch.Tensor, R: float, s: float) -> int:
    """Steps 3/4: the first token whose inclusive cumulative mass exceeds s*R."""
    lib = _load()
    r = _cpu(r, torch.float64).contiguous()
    return int(lib.oracle_inverse_cdf(_ptr(r), r.numel(), float(R), float(s), None, None))


@dataclass
class SampleResult:
    accepted_len: torch.Tensor   # [B] int32
    out_tokens: torch.Tensor     # [TQ] int32
    rho: torch.Tensor            # [TD] float64, NaN for drafts after the first rejection
    resid_mass: torch.Tensor     # [B] float64
    cdf_lo: torch.Tensor         # [B] float64
    cdf_hi: torch.Tensor         # [B] float64
    flags: torch.Tensor          # [B] int32
    status: int                  # OK, ERR_TOKEN or ERR_PARAM
    margin: Optional[torch.Tensor] = None   # [B] float64: smallest top-p decision margin (filtered calls only)


def rejection_sample(target_logits: torch.Tensor, draft_logits: torch.Tensor,
                     draft_ids: torch.Tensor, q_indptr: torch.Tensor, u_accept: torch.Tensor,
                     u_sample: torch.Tensor, vocab: Optional[int] = None,
                     temperature: Optional[torch.Tensor] = None, top_k: Optional[torch.Tensor] = None,
                     top_p: Optional[torch.Tensor] = None) -> SampleResult:
    """Speculative rejection sampling for the whole batch, in float64, one request at a time.
    ``temperature`` ([B] float32, optional): > 0 verifies at that temperature, 0 verifies greedily."""
    lib = _load()
    tl = _cpu(target_logits)
    dl = _cpu(draft_logits)
    assert tl.dim() == 2 and tl.stride(1) == 1
    dt = _dtype_code(tl)
    row_stride = tl.stride(0)
    V = int(vocab if vocab is not None else tl.shape[1])
    if dl.numel() > 0:
        assert dl.dim() == 2 and dl.stride(1) == 1 and dl.stride(0) == row_stride
        assert _dtype_code(dl) == dt
    qi = _cpu(q_indptr, torch.int32).contiguous()
    B = qi.numel() - 1
    TQ = int(qi[-1])
    TD = TQ - B
    ids = _cpu(draft_ids, torch.int32).contiguous()
    ua = _cpu(u_accept, torch.float32).contiguous()
    us = _cpu(u_sample, torch.float32).contiguous()
    assert ids.numel() == TD and ua.numel() == TD and us.numel() == B
    res = SampleResult(
        accepted_len=torch.empty(B, dtype=torch.int32),
        out_tokens=torch.empty(TQ, dtype=torch.int32),
        rho=torch.empty(TD, dtype=torch.float64),
        resid_mass=torch.empty(B, dtype=torch.float64),
        cdf_lo=torch.empty(B, dtype=torch.float64),
        cdf_hi=torch.empty(B, dtype=torch.float64),
        flags=torch.empty(B, dtype=torch.int32),
        status=OK)
    if top_k is not None or top_p is not None:
        tau = _cpu(temperature, torch.float32).contiguous() if temperature is not None else None
        tk = _cpu(top_k, torch.int32).contiguous() if top_k is not None else None
        tp = _cpu(top_p, torch.float32).contiguous() if top_p is not None else None
        res.margin = torch.empty(B, dtype=torch.float64)
        lib.oracle_rejection_sample_filtered.restype = c.c_int
        lib.oracle_rejection_sample_filtered.argtypes = [c.c_int32, c.c_int64, c.c_int64, c.c_int32] + [c.c_void_p] * 17
        st = lib.oracle_rejection_sample_filtered(
            B, V, row_stride, dt, _ptr(tl), _ptr(dl), _ptr(ids), _ptr(qi), _ptr(ua), _ptr(us), _ptr(tau), _ptr(tk),
            _ptr(tp), _ptr(res.accepted_len), _ptr(res.out_tokens), _ptr(res.rho), _ptr(res.resid_mass),
            _ptr(res.cdf_lo), _ptr(res.cdf_hi), _ptr(res.flags), _ptr(res.margin))
    elif temperature is None:
        st = lib.oracle_rejection_sample(
            B, V, row_stride, dt, _ptr(tl), _ptr(dl), _ptr(ids), _ptr(qi), _ptr(ua), _ptr(us),
            _ptr(res.accepted_len), _ptr(res.out_tokens), _ptr(res.rho), _ptr(res.resid_mass),
            _ptr(res.cdf_lo), _ptr(res.cdf_hi), _ptr(res.flags))
    else:
        tau = _cpu(temperature, torch.float32).contiguous()
        assert tau.numel() == B
        lib.oracle_rejection_sample_tau.restype = c.c_int
        lib.oracle_rejection_sample_tau.argtypes = [c.c_int32, c.c_int64, c.c_int64, c.c_int32] + [c.c_void_p] * 14
        st = lib.oracle_rejection_sample_tau(
            B, V, row_stride, dt, _ptr(tl), _ptr(dl), _ptr(ids), _ptr(qi), _ptr(ua), _ptr(us), _ptr(tau),
            _ptr(res.accepted_len), _ptr(res.out_tokens), _ptr(res.rho), _ptr(res.resid_mass),
            _ptr(res.cdf_lo), _ptr(res.cdf_hi), _ptr(res.flags))
    if st not in (OK, ERR_TOKEN, ERR_PARAM):
        raise OracleError(st)
    res.status = st
    return res


def emit_cdf(r: int, n: int, target_logits: torch.Tensor, draft_logits: torch.Tensor,
             q_indptr: torch.Tensor, vocab: Optional[int] = None, tau: float = 1.0, top_k: int = 0,
             top_p: float = 1.0):
    """Inclusive cumulative distribution request ``r``'s emitted token was drawn from, and R."""
    lib = _load()
    tl = _cpu(target_logits)
    dl = _cpu(draft_logits)
    V = int(vocab if vocab is not None else tl.shape[1])
    qi = _cpu(q_indptr, torch.int32).contiguous()
    cdf = torch.empty(V, dtype=torch.float64)
    lib.oracle_emit_cdf_filtered.restype = c.c_double
    lib.oracle_emit_cdf_filtered.argtypes = [c.c_int32, c.c_int32, c.c_int64, c.c_int64, c.c_int32, c.c_void_p, c.c_void_p,
                                             c.c_void_p, c.c_double, c.c_int32, c.c_double, c.c_void_p]
    R = lib.oracle_emit_cdf_filtered(int(r), int(n), V, tl.stride(0), _dtype_code(tl), _ptr(tl), _ptr(dl),
                                     _ptr(qi), float(tau), int(top_k), float(top_p), _ptr(cdf))
    return cdf, float(R)


def kv_append(new_k: torch.Tensor, new_v: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
              kv_strides: Sequence[int], block_table: torch.Tensor, seq_lens: torch.Tensor, q_indptr: torch.Tensor,
              page_size: int, num_pages: int, rope_base: float = 0.0) -> None:
    """Write the new positions' K/V ([TQ, Hkv, D]) into their pages, in place (bit copies).  With
    rope_base > 0 the K rows are rotated to their absolute positions first (V is not)."""
    lib = _load()
    nk, nv = _cpu(new_k).contiguous(), _cpu(new_v).contiguous()
    if rope_base > 0.0:
        nk = round_to(rope(nk, new_positions(seq_lens, q_indptr), rope_base), nk.dtype).contiguous()
    assert nk.dtype == k_cache.dtype == v_cache.dtype == nv.dtype
    _dtype_code(nk)
    TQ, Hkv, D = nk.shape
    bt = _cpu(block_table, torch.int32).contiguous()
    sl = _cpu(seq_lens, torch.int32).contiguous()
    qi = _cpu(q_indptr, torch.int32).contiguous()
    st = lib.oracle_kv_append(sl.numel(), Hkv, D, page_size, num_pages, bt.shape[1], nk.element_size(), _ptr(nk),
                              _ptr(nv), _ptr(_cpu(k_cache)), _ptr(_cpu(v_cache)), int(kv_strides[0]),
                              int(kv_strides[1]), int(kv_strides[2]), _ptr(bt), _ptr(sl), _ptr(qi))
    if st != OK:
        raise OracleError(st)


def rope(x: torch.Tensor, positions: torch.Tensor, base: float) -> torch.Tensor:
    """Rotary embedding of x [rows, H, D] at the given absolute positions; float64 result."""
    lib = _load()
    xc = _cpu(x).contiguous()
    rows, H, D = xc.shape
    pos = _cpu(positions, torch.int32).contiguous()
    assert pos.numel() == rows
    out = torch.empty(rows, H, D, dtype=torch.float64)
    lib.oracle_rope_rows.argtypes = [c.c_void_p, c.c_int32, c.c_int64, c.c_int32, c.c_int32, c.c_void_p, c.c_double,
                                     c.c_void_p]
    st = lib.oracle_rope_rows(_ptr(xc), _dtype_code(xc), rows, H, D, _ptr(pos), float(base), _ptr(out))
    if st != OK:
        raise OracleError(st)
    return out


def new_positions(seq_lens: torch.Tensor, q_indptr: torch.Tensor) -> torch.Tensor:
    """Absolute position of every new row: row q_indptr[r]+j is token L_r-(k_r+1)+j of request r."""
    sl, qi = _cpu(seq_lens, torch.int32).tolist(), _cpu(q_indptr, torch.int32).tolist()
    pos = torch.empty(qi[-1], dtype=torch.int32)
    for r, L in enumerate(sl):
        m = qi[r + 1] - qi[r]
        for j in range(m):
            pos[qi[r] + j] = L - m + j
    return pos


def round_to(x64: torch.Tensor, dtype: torch.dtype) -> torch.Tensor:
    """double -> binary32 -> dtype, each step round-to-nearest-even (what the CUDA path does)."""
    return x64.to(torch.float32).to(dtype)


def kv_rollback(seq_lens: torch.Tensor, q_indptr: torch.Tensor, accepted_len: torch.Tensor) -> torch.Tensor:
    """Lengths after dropping the rejected drafts: L - (k - n)."""
    lib = _load()
    sl = _cpu(seq_lens, torch.int32).contiguous()
    qi = _cpu(q_indptr, torch.int32).contiguous()
    al = _cpu(accepted_len, torch.int32).contiguous()
    out = torch.empty_like(sl)
    st = lib.oracle_kv_rollback(sl.numel(), _ptr(sl), _ptr(qi), _ptr(al), _ptr(out))
    if st != OK:
        raise OracleError(st)
    return out


def draft_confidence(draft_logits: torch.Tensor, draft_ids: Optional[torch.Tensor], q_indptr: torch.Tensor,
                     vocab: Optional[int] = None):
    """Per-draft top-1 probability, probability of the drafted token (None without ids) and the
    per-request product of the top-1 probabilities, all float64."""
    lib = _load()
    dl = _cpu(draft_logits)
    qi = _cpu(q_indptr, torch.int32).contiguous()
    B = qi.numel() - 1
    TD = int(qi[-1]) - B
    V = int(vocab if vocab is not None else dl.shape[1])
    ids = _cpu(draft_ids, torch.int32).contiguous() if draft_ids is not None else None
    cmax = torch.empty(TD, dtype=torch.float64)
    ctok = torch.empty(TD, dtype=torch.float64) if ids is not None else None
    creq = torch.empty(B, dtype=torch.float64)
    lib.oracle_draft_confidence.restype = c.c_int
    lib.oracle_draft_confidence.argtypes = [c.c_int32, c.c_int64, c.c_int64, c.c_int32] + [c.c_void_p] * 6
    st = lib.oracle_draft_confidence(B, V, dl.stride(0) if dl.dim() == 2 and dl.numel() else V, _dtype_code(dl), _ptr(dl),
                                     _ptr(ids), _ptr(qi), _ptr(cmax), _ptr(ctok), _ptr(creq))
    if st not in (OK, ERR_TOKEN):
        raise OracleError(st)
    return cmax, ctok, creq


def select_speculation(confidence: torch.Tensor, k_in: torch.Tensor, alpha: float):
    """Keep-top-(1-alpha): returns (k_out [B] int32, n_drop)."""
    lib = _load()
    conf = _cpu(confidence, torch.float32).contiguous()
    kin = _cpu(k_in, torch.int32).contiguous()
    assert conf.numel() == kin.numel()
    kout = torch.empty_like(kin)
    nd = c.c_int32(0)
    lib.oracle_select_speculation.restype = c.c_int
    lib.oracle_select_speculation.argtypes = [c.c_int32, c.c_void_p, c.c_void_p, c.c_double, c.c_void_p, c.c_void_p]
    st = lib.oracle_select_speculation(kin.numel(), _ptr(conf), _ptr(kin), float(alpha), _ptr(kout), c.byref(nd))
    if st != OK:
        raise OracleError(st)
    return kout, int(nd.value)


# ---- the paper's scheduler numerics (Eq. 1-4, the gain G, Algorithm 1) ----

def sp_recurrence(B: float, N: int, theta: float, T: int):
    """Eq. 1 iterated from Appendix A.1's initial conditions: (s_a, s_r, n), each [T+1] float64."""
    lib = _load()
    sa, sr, n = (torch.empty(T + 1, dtype=torch.float64) for _ in range(3))
    lib.oracle_sp_recurrence.restype = c.c_int
    lib.oracle_sp_recurrence.argtypes = [c.c_double, c.c_int32, c.c_double, c.c_int32, c.c_void_p, c.c_void_p, c.c_void_p]
    st = lib.oracle_sp_recurrence(float(B), int(N), float(theta), int(T), _ptr(sa), _ptr(sr), _ptr(n))
    if st != OK:
        raise OracleError(st)
    return sa, sr, n


def sp_effective_batch(B: float, N: int, theta: float) -> float:
    lib = _load()
    lib.oracle_sp_effective_batch.restype = c.c_double
    lib.oracle_sp_effective_batch.argtypes = [c.c_double, c.c_int32, c.c_double]
    return float(lib.oracle_sp_effective_batch(float(B), int(N), float(theta)))


def alpha_recurrence(B: float, N: int, alpha: float, T: int) -> torch.Tensor:
    lib = _load()
    bt = torch.empty(T + 1, dtype=torch.float64)
    lib.oracle_alpha_recurrence.restype = c.c_int
    lib.oracle_alpha_recurrence.argtypes = [c.c_double, c.c_int32, c.c_double, c.c_int32, c.c_void_p]
    st = lib.oracle_alpha_recurrence(float(B), int(N), float(alpha), int(T), _ptr(bt))
    if st != OK:
        raise OracleError(st)
    return bt


def alpha_batch(B: float, N: int, alpha: float) -> float:
    lib = _load()
    lib.oracle_alpha_batch.restype = c.c_double
    lib.oracle_alpha_batch.argtypes = [c.c_double, c.c_int32, c.c_double]
    return float(lib.oracle_alpha_batch(float(B), int(N), float(alpha)))


def alpha_effective_batch(B: float, N: int, alpha: float, theta_alpha: float) -> float:
    lib = _load()
    lib.oracle_alpha_effective_batch.restype = c.c_double
    lib.oracle_alpha_effective_batch.argtypes = [c.c_double, c.c_int32, c.c_double, c.c_double]
    return float(lib.oracle_alpha_effective_batch(float(B), int(N), float(alpha), float(theta_alpha)))


def delay_gain(I: float, pdr: float, bs: float, i_delay: float, i_wait: Sequence[float]) -> float:
    lib = _load()
    w = torch.tensor(list(i_wait), dtype=torch.float64)
    lib.oracle_delay_gain.restype = c.c_double
    lib.oracle_delay_gain.argtypes = [c.c_double, c.c_int32, c.c_double, c.c_double, c.c_double, c.c_void_p]
    return float(lib.oracle_delay_gain(float(I), w.numel(), float(pdr), float(bs), float(i_delay), _ptr(w)))


def lookahead_memory(ell: torch.Tensor, tau: torch.Tensor, prec: torch.Tensor, pp: int, theta: float,
                     horizon: int = 64) -> torch.Tensor:
    """Algorithm 1: estimated KV memory (tokens) at look-ahead iterations 1..horizon, float64."""
    lib = _load()
    ell = _cpu(ell, torch.int32).contiguous()
    tau = _cpu(tau, torch.int32).contiguous()
    prec = _cpu(prec, torch.float64).contiguous()
    assert ell.numel() == tau.numel() == prec.numel()
    M = torch.empty(horizon, dtype=torch.float64)
    lib.oracle_lookahead_memory.restype = c.c_int
    lib.oracle_lookahead_memory.argtypes = [c.c_int32, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int32, c.c_double,
                                            c.c_int32, c.c_void_p]
    st = lib.oracle_lookahead_memory(ell.numel(), _ptr(ell), _ptr(tau), _ptr(prec), int(pp), float(theta), int(horizon),
                                     _ptr(M))
    if st != OK:
        raise OracleError(st)
    return M


def filtered_row(logits_row: torch.Tensor, tau: float = 1.0, top_k: int = 0, top_p: float = 1.0):
    """Step 1 under top-k / top-p: (p [V] float64, kept count, top-p decision margin)."""
    lib = _load()
    row = _cpu(logits_row).contiguous()
    V = row.numel()
    p = torch.empty(V, dtype=torch.float64)
    scratch = torch.empty(V, dtype=torch.float64)
    m = c.c_double(0.0)
    lib.oracle_filtered_row.restype = c.c_int64
    lib.oracle_filtered_row.argtypes = [c.c_void_p, c.c_int32, c.c_int64, c.c_int64, c.c_double, c.c_int32, c.c_double,
                                        c.c_void_p, c.c_void_p, c.c_void_p]
    kept = lib.oracle_filtered_row(_ptr(row), _dtype_code(row), 0, V, float(tau), int(top_k), float(top_p), _ptr(p),
                                   _ptr(scratch), c.byref(m))
    return p, int(kept), float(m.value)


def lm_head(hidden: torch.Tensor, weight: torch.Tensor, v_begin: int = 0, v_end: Optional[int] = None) -> torch.Tensor:
    """logits[:, v_begin:v_end] = hidden @ weight[v_begin:v_end].T in float64 (plain loops)."""
    lib = _load()
    h = _cpu(hidden).contiguous()
    w = _cpu(weight).contiguous()
    assert h.dim() == 2 and w.dim() == 2 and h.shape[1] == w.shape[1] and _dtype_code(h) == _dtype_code(w)
    V = w.shape[0]
    v_end = V if v_end is None else int(v_end)
    out = torch.empty((h.shape[0], v_end - int(v_begin)), dtype=torch.float64)
    lib.oracle_lm_head.restype = c.c_int
    lib.oracle_lm_head.argtypes = [c.c_int32, c.c_int32, c.c_int64, c.c_int32, c.c_void_p, c.c_void_p, c.c_int64, c.c_int64,
                                   c.c_void_p]
    st = lib.oracle_lm_head(h.shape[0], h.shape[1], V, _dtype_code(h), _ptr(h), _ptr(w), int(v_begin), v_end, _ptr(out))
    if st != OK:
        raise OracleError(st)
    return out
