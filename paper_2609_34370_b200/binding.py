"""ctypes binding of include/spx.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Tuple

import torch

from .build import LIB_PATH

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA = 0, 1, 2, 3, 4
DEV_BAD_PAGE, DEV_BAD_TOKEN, DEV_BAD_LEN, DEV_TIMEOUT, DEV_DEGENERATE, DEV_BAD_PARAM = 1, 2, 4, 8, 16, 32
BF16, F32 = 0, 1

EXPORTS = ("spx_workspace_size", "spx_verify_attention", "spx_rejection_sample", "spx_verify_step",
           "spx_host_step_arena_size", "spx_verify_step_host", "spx_status_string", "spx_last_launch_count",
           "spx_set_timing_events", "spx_plan_layout", "spx_debug_timeline", "spx_debug_wait_expiry", "spx_rejection_sample_static", "spx_kv_append", "spx_kv_rollback",
           "spx_draft_confidence_workspace", "spx_draft_confidence", "spx_select_speculation",
           "spx_lookahead_memory", "spx_sp_effective_batch", "spx_selective_batch", "spx_selective_effective_batch",
           "spx_delay_gain", "spx_lm_head")


class AttnArgs(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("total_q", C.c_int32), ("max_q_len", C.c_int32),
        ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("page_size", C.c_int32), ("num_pages", C.c_int32), ("max_pages_per_req", C.c_int32),
        ("kv_dtype", C.c_int), ("sm_scale", C.c_float),
        ("q", C.c_void_p), ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
        ("kv_stride_page", C.c_int64), ("kv_stride_head", C.c_int64), ("kv_stride_token", C.c_int64),
        ("block_table", C.c_void_p), ("seq_lens", C.c_void_p), ("q_indptr", C.c_void_p),
        ("out", C.c_void_p), ("lse", C.c_void_p),
    ]


class SampleArgs(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("total_q", C.c_int32), ("vocab", C.c_int32),
        ("logits_row_stride", C.c_int64), ("logits_dtype", C.c_int),
        ("target_logits", C.c_void_p), ("draft_logits", C.c_void_p), ("draft_token_ids", C.c_void_p),
        ("q_indptr", C.c_void_p), ("u_accept", C.c_void_p), ("u_sample", C.c_void_p),
        ("accepted_len", C.c_void_p), ("out_tokens", C.c_void_p), ("diag_ratio", C.c_void_p),
        ("temperature", C.c_void_p), ("top_k", C.c_void_p), ("top_p", C.c_void_p), ("target_tile_stats", C.c_void_p),
    ]


class KvAppendArgs(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("total_q", C.c_int32),
        ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("page_size", C.c_int32), ("num_pages", C.c_int32),
        ("max_pages_per_req", C.c_int32), ("kv_dtype", C.c_int),
        ("new_k", C.c_void_p), ("new_v", C.c_void_p), ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
        ("kv_stride_page", C.c_int64), ("kv_stride_head", C.c_int64), ("kv_stride_token", C.c_int64),
        ("block_table", C.c_void_p), ("seq_lens", C.c_void_p), ("q_indptr", C.c_void_p),
        ("rope_base", C.c_float), ("num_q_heads", C.c_int32), ("q_rows", C.c_void_p),
    ]


class ConfArgs(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("total_q", C.c_int32), ("vocab", C.c_int32), ("logits_row_stride", C.c_int64),
        ("logits_dtype", C.c_int),
        ("draft_logits", C.c_void_p), ("draft_token_ids", C.c_void_p), ("q_indptr", C.c_void_p),
        ("conf_max", C.c_void_p), ("conf_tok", C.c_void_p), ("req_conf", C.c_void_p),
    ]


class LmHeadArgs(C.Structure):
    _fields_ = [
        ("rows", C.c_int32), ("hidden_dim", C.c_int32), ("vocab", C.c_int32),
        ("hidden", C.c_void_p), ("weight", C.c_void_p), ("logits", C.c_void_p), ("logits_row_stride", C.c_int64),
        ("tile_stats", C.c_void_p),
    ]


class SpxError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"libspx: {what} (status {code})")
        self.code = code


_lib = None


def lib_path() -> str:
    return LIB_PATH


def load_library():
    """Load libspx.so; raises if it has not been built (there is no other implementation)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise SpxError(-1, f"{LIB_PATH} is missing: run paper_2609_34370_b200.build.build() "
                               "(or __graft_entry__.build()) first")
        lib = C.CDLL(LIB_PATH)
        lib.spx_workspace_size.restype = C.c_size_t
        lib.spx_workspace_size.argtypes = [C.POINTER(AttnArgs), C.POINTER(SampleArgs)]
        for name in ("spx_verify_attention", "spx_rejection_sample"):
            fn = getattr(lib, name)
            fn.restype = C.c_int
            fn.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        lib.spx_verify_step.restype = C.c_int
        lib.spx_verify_step.argtypes = [C.POINTER(AttnArgs), C.POINTER(SampleArgs), C.c_void_p, C.c_size_t,
                                        C.c_void_p, C.c_void_p]
        lib.spx_host_step_arena_size.restype = C.c_size_t
        lib.spx_host_step_arena_size.argtypes = [C.POINTER(AttnArgs), C.POINTER(SampleArgs), C.c_int64]
        lib.spx_verify_step_host.restype = C.c_int
        lib.spx_verify_step_host.argtypes = [C.POINTER(AttnArgs), C.POINTER(SampleArgs), C.c_int64, C.c_void_p,
                                             C.c_size_t, C.c_void_p, C.c_void_p]
        lib.spx_status_string.restype = C.c_char_p
        lib.spx_status_string.argtypes = [C.c_int]
        lib.spx_last_launch_count.restype = C.c_int32
        lib.spx_plan_layout.restype = C.c_int
        lib.spx_debug_timeline.restype = C.c_int
        lib.spx_debug_timeline.argtypes = [C.c_void_p, C.c_int64, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        lib.spx_plan_layout.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
        lib.spx_debug_wait_expiry.restype = C.c_int
        lib.spx_debug_wait_expiry.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        lib.spx_rejection_sample_static.restype = C.c_int
        lib.spx_rejection_sample_static.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        lib.spx_kv_append.restype = C.c_int
        lib.spx_kv_append.argtypes = [C.POINTER(KvAppendArgs), C.c_void_p, C.c_void_p]
        lib.spx_kv_rollback.restype = C.c_int
        lib.spx_kv_rollback.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.spx_draft_confidence_workspace.restype = C.c_size_t
        lib.spx_draft_confidence_workspace.argtypes = [C.POINTER(ConfArgs)]
        lib.spx_draft_confidence.restype = C.c_int
        lib.spx_draft_confidence.argtypes = [C.POINTER(ConfArgs), C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        lib.spx_select_speculation.restype = C.c_int
        lib.spx_select_speculation.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_double, C.c_void_p, C.c_void_p,
                                               C.c_void_p, C.c_void_p]
        lib.spx_lookahead_memory.restype = C.c_int
        lib.spx_lookahead_memory.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_double, C.c_int32,
                                             C.c_void_p, C.c_void_p]
        for name, nargs in (("spx_sp_effective_batch", 0), ("spx_selective_batch", 0), ("spx_selective_effective_batch", 1)):
            fn = getattr(lib, name)
            fn.restype = C.c_double
            fn.argtypes = [C.c_double, C.c_int32, C.c_double] + [C.c_double] * nargs
        lib.spx_delay_gain.restype = C.c_double
        lib.spx_delay_gain.argtypes = [C.c_double, C.c_int32, C.c_double, C.c_double, C.c_double, C.POINTER(C.c_double)]
        lib.spx_lm_head.restype = C.c_int
        lib.spx_lm_head.argtypes = [C.POINTER(LmHeadArgs), C.c_void_p, C.c_void_p]
        lib.spx_set_timing_events.restype = None
        lib.spx_set_timing_events.argtypes = [C.c_void_p, C.c_void_p]
        _lib = lib
    return _lib


def exported_symbols() -> Tuple[str, ...]:
    return EXPORTS


def _check(code: int):
    if code != OK:
        raise SpxError(code, load_library().spx_status_string(code).decode())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"bf16 or fp32 expected, got {t.dtype}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None or t.numel() == 0 else t.data_ptr()


def _stream(device) -> int:
    return torch.cuda.current_stream(device).cuda_stream


def _require_cuda(*tensors):
    for t in tensors:
        if t is not None and t.device.type != "cuda":
            raise SpxError(ERR_INVALID_ARG, "device tensors required (there is no CPU path)")


def make_attn_args(q, k_cache, v_cache, kv_strides, block_table, seq_lens, q_indptr, num_kv_heads, page_size,
                   num_pages, out, lse=None, sm_scale=0.0, max_q_len=0) -> AttnArgs:
    TQ, Hq, D = q.shape
    a = AttnArgs()
    a.batch = seq_lens.numel()
    a.total_q = TQ
    a.max_q_len = max_q_len
    a.num_q_heads, a.num_kv_heads, a.head_dim, a.page_size = Hq, num_kv_heads, D, page_size
    a.num_pages = num_pages
    a.max_pages_per_req = block_table.shape[1] if block_table.dim() == 2 else 0
    a.kv_dtype = _dtype_code(q)
    a.sm_scale = sm_scale
    a.q, a.k_cache, a.v_cache = _ptr(q), _ptr(k_cache), _ptr(v_cache)
    a.kv_stride_page, a.kv_stride_head, a.kv_stride_token = (int(x) for x in kv_strides)
    a.block_table, a.seq_lens, a.q_indptr = _ptr(block_table), _ptr(seq_lens), q_indptr.data_ptr()
    a.out, a.lse = _ptr(out), _ptr(lse)
    return a


def make_sample_args(target_logits, draft_logits, draft_ids, q_indptr, u_accept, u_sample, accepted_len,
                     out_tokens, diag_ratio=None, vocab=None, temperature=None, top_k=None, top_p=None,
                     target_tile_stats=None) -> SampleArgs:
    s = SampleArgs()
    s.batch = q_indptr.numel() - 1
    s.total_q = target_logits.shape[0]
    s.vocab = int(vocab if vocab is not None else target_logits.shape[1])
    s.logits_row_stride = target_logits.stride(0)
    s.logits_dtype = _dtype_code(target_logits)
    s.target_logits, s.draft_logits = _ptr(target_logits), _ptr(draft_logits)
    s.draft_token_ids, s.q_indptr = _ptr(draft_ids), q_indptr.data_ptr()
    s.u_accept, s.u_sample = _ptr(u_accept), _ptr(u_sample)
    s.accepted_len, s.out_tokens, s.diag_ratio = _ptr(accepted_len), _ptr(out_tokens), _ptr(diag_ratio)
    s.temperature, s.top_k, s.top_p = _ptr(temperature), _ptr(top_k), _ptr(top_p)
    s.target_tile_stats = _ptr(target_tile_stats)
    return s


def workspace_size(attn: Optional[AttnArgs], sample: Optional[SampleArgs]) -> int:
    lib = load_library()
    n = lib.spx_workspace_size(C.byref(attn) if attn is not None else None,
                               C.byref(sample) if sample is not None else None)
    if n == 0:
        raise SpxError(ERR_INVALID_ARG, "invalid arguments for workspace sizing")
    return int(n)


@dataclass
class Workspace:
    """Caller-owned scratch and status word (torch is used for the allocation only)."""
    buf: torch.Tensor
    status: torch.Tensor

    @staticmethod
    def allocate(nbytes: int, device) -> "Workspace":
        return Workspace(torch.empty(nbytes, dtype=torch.uint8, device=device),
                         torch.zeros(1, dtype=torch.int32, device=device))

    def ensure(self, nbytes: int):
        if self.buf.numel() < nbytes:
            self.buf = torch.empty(nbytes, dtype=torch.uint8, device=self.buf.device)


def verify_attention(q, k_cache, v_cache, kv_strides, block_table, seq_lens, q_indptr, num_kv_heads, page_size,
                     num_pages, out=None, lse=None, sm_scale=0.0, max_q_len=0, ws: Optional[Workspace] = None,
                     want_lse=True):
    """spx_verify_attention on the current stream.  Returns (out, lse, ws)."""
    _require_cuda(q, k_cache, v_cache, block_table, seq_lens, q_indptr)
    lib = load_library()
    if out is None:
        out = torch.empty_like(q)
    if lse is None and want_lse:
        lse = torch.empty(q.shape[:2], dtype=torch.float32, device=q.device)
    a = make_attn_args(q, k_cache, v_cache, kv_strides, block_table, seq_lens, q_indptr, num_kv_heads, page_size,
                       num_pages, out, lse, sm_scale, max_q_len)
    need = workspace_size(a, None)
    if ws is None:
        ws = Workspace.allocate(need, q.device)
    ws.ensure(need)
    _check(lib.spx_verify_attention(C.byref(a), ws.buf.data_ptr(), ws.buf.numel(), ws.status.data_ptr(),
                                    _stream(q.device)))
    return out, lse, ws


def rejection_sample(target_logits, draft_logits, draft_ids, q_indptr, u_accept, u_sample, vocab=None,
                     want_ratio=False, ws: Optional[Workspace] = None, temperature=None, top_k=None, top_p=None,
                     target_tile_stats=None, accepted=None, tokens=None):
    """spx_rejection_sample on the current stream.  Returns (accepted_len, out_tokens, ratio, ws).
    ``temperature`` ([B] float32 on the device, optional) selects the verification variant per request;
    ``accepted`` ([B] int32) and ``tokens`` ([TQ] int32) are the output buffers if the caller brings its own."""
    _require_cuda(target_logits, draft_logits, draft_ids, q_indptr, u_accept, u_sample)
    for extra in (temperature, top_k, top_p):
        if extra is not None:
            _require_cuda(extra)
    lib = load_library()
    dev = target_logits.device
    B = q_indptr.numel() - 1
    TQ = target_logits.shape[0]
    if accepted is None:
        accepted = torch.empty(B, dtype=torch.int32, device=dev)
    if tokens is None:
        tokens = torch.empty(TQ, dtype=torch.int32, device=dev)
    ratio = torch.empty(TQ - B, dtype=torch.float32, device=dev) if want_ratio else None
    s = make_sample_args(target_logits, draft_logits, draft_ids, q_indptr, u_accept, u_sample, accepted, tokens,
                         ratio, vocab, temperature, top_k, top_p, target_tile_stats)
    need = workspace_size(None, s)
    if ws is None:
        ws = Workspace.allocate(need, dev)
    ws.ensure(need)
    _check(lib.spx_rejection_sample(C.byref(s), ws.buf.data_ptr(), ws.buf.numel(), ws.status.data_ptr(),
                                    _stream(dev)))
    return accepted, tokens, ratio, ws


def verify_step(attn: AttnArgs, sample: SampleArgs, ws: Workspace, device):
    """spx_verify_step with prebuilt argument structs (the benchmark's hot call)."""
    lib = load_library()
    _check(lib.spx_verify_step(C.byref(attn), C.byref(sample), ws.buf.data_ptr(), ws.buf.numel(),
                               ws.status.data_ptr(), _stream(device)))


def verify_step_host(attn: AttnArgs, sample: SampleArgs, kv_pool_elems: int, arena: torch.Tensor,
                     status_host: torch.Tensor, device):
    """spx_verify_step_host: every pointer in the structs is a host pointer."""
    lib = load_library()
    _check(lib.spx_verify_step_host(C.byref(attn), C.byref(sample), int(kv_pool_elems), arena.data_ptr(),
                                    arena.numel(), status_host.data_ptr(), _stream(device)))


def host_step_arena_size(attn: AttnArgs, sample: SampleArgs, kv_pool_elems: int) -> int:
    n = load_library().spx_host_step_arena_size(C.byref(attn), C.byref(sample), int(kv_pool_elems))
    if n == 0:
        raise SpxError(ERR_INVALID_ARG, "invalid arguments for arena sizing")
    return int(n)


def plan_layout(attn_args) -> dict:
    """spx_plan_layout: byte offsets of the attention work plan inside the workspace."""
    out = (C.c_int64 * 8)()
    _check(load_library().spx_plan_layout(C.byref(attn_args), out))
    keys = ("header", "cta_off", "work", "max_work", "pair_nchunks", "pair_part_base", "max_part_slots", "attn_bytes")
    return dict(zip(keys, (int(v) for v in out)))


def debug_timeline():
    """spx_debug_timeline: numpy uint64 [kernels, ctas, 4] = (start ns, end ns, SM id, 0) of the most
    recent launches.  Only a timeline build of the library records them (SpxError otherwise)."""
    import numpy as np
    lib = load_library()
    nk, nc = C.c_int32(0), C.c_int32(0)
    lib.spx_debug_timeline(None, 0, C.byref(nk), C.byref(nc))
    out = np.zeros((nk.value, nc.value, 4), dtype=np.uint64)
    _check(lib.spx_debug_timeline(out.ctypes.data, out.size, C.byref(nk), C.byref(nc)))
    return out


def last_launch_count() -> int:
    return int(load_library().spx_last_launch_count())


def set_timing_events(start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event]):
    """Record `start`/`stop` around the verify-attention kernel of later calls (None, None clears).

    The events must have been recorded once already so that their CUDA handles exist.
    """
    lib = load_library()
    if start is None or stop is None:
        lib.spx_set_timing_events(None, None)
    else:
        lib.spx_set_timing_events(start.cuda_event, stop.cuda_event)


STATIC_SCRATCH_BYTES = 4 << 20


def rejection_sample_static(target_logits, draft_logits, draft_ids, q_indptr, u_accept, u_sample, vocab=None,
                            status: Optional[torch.Tensor] = None):
    """spx_rejection_sample_static on the current stream: the sampling half for callers that can
    neither allocate nor pass a workspace (the scratch is a fixed array inside the library).

    Only the outputs and, if none is given, the status word are allocated here, by torch, on the
    caller's side of the boundary; the library call itself allocates nothing.  Returns
    (accepted_len, out_tokens, status).  Raises SpxError(ERR_WORKSPACE) when the batch needs more
    than STATIC_SCRATCH_BYTES of scratch.
    """
    _require_cuda(target_logits, draft_logits, draft_ids, q_indptr, u_accept, u_sample)
    lib = load_library()
    dev = target_logits.device
    B = q_indptr.numel() - 1
    accepted = torch.empty(B, dtype=torch.int32, device=dev)
    tokens = torch.empty(target_logits.shape[0], dtype=torch.int32, device=dev)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    s = make_sample_args(target_logits, draft_logits, draft_ids, q_indptr, u_accept, u_sample, accepted, tokens,
                         None, vocab)
    _check(lib.spx_rejection_sample_static(C.byref(s), status.data_ptr(), _stream(dev)))
    return accepted, tokens, status


def kv_append(new_k, new_v, k_cache, v_cache, kv_strides, block_table, seq_lens, q_indptr, page_size, num_pages,
              status: Optional[torch.Tensor] = None, rope_base: float = 0.0, q_rows: Optional[torch.Tensor] = None):
    """spx_kv_append on the current stream: the new positions' K/V go into their pages, in place.
    rope_base > 0: the K rows (and q_rows [TQ, Hq, D], in place) are rotated to their positions."""
    _require_cuda(new_k, new_v, k_cache, v_cache, block_table, seq_lens, q_indptr)
    lib = load_library()
    dev = new_k.device
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    a = KvAppendArgs()
    a.batch, a.total_q = seq_lens.numel(), new_k.shape[0]
    a.num_kv_heads, a.head_dim, a.page_size, a.num_pages = new_k.shape[1], new_k.shape[2], page_size, num_pages
    a.max_pages_per_req = block_table.shape[1]
    a.kv_dtype = _dtype_code(new_k)
    a.new_k, a.new_v, a.k_cache, a.v_cache = _ptr(new_k), _ptr(new_v), _ptr(k_cache), _ptr(v_cache)
    a.kv_stride_page, a.kv_stride_head, a.kv_stride_token = (int(x) for x in kv_strides)
    a.block_table, a.seq_lens, a.q_indptr = _ptr(block_table), _ptr(seq_lens), q_indptr.data_ptr()
    a.rope_base = float(rope_base)
    if q_rows is not None:
        _require_cuda(q_rows)
        if q_rows.dtype != new_k.dtype or not q_rows.is_contiguous():
            raise SpxError(ERR_INVALID_ARG, "q_rows must be contiguous and of the cache's dtype")
        a.num_q_heads, a.q_rows = q_rows.shape[1], _ptr(q_rows)
    _check(lib.spx_kv_append(C.byref(a), status.data_ptr(), _stream(dev)))
    return status


def kv_rollback(seq_lens, q_indptr, accepted_len, out: Optional[torch.Tensor] = None,
                status: Optional[torch.Tensor] = None):
    """spx_kv_rollback on the current stream.  Returns (new_seq_lens, status)."""
    _require_cuda(seq_lens, q_indptr, accepted_len)
    lib = load_library()
    dev = seq_lens.device
    if out is None:
        out = torch.empty_like(seq_lens)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    _check(lib.spx_kv_rollback(seq_lens.numel(), seq_lens.data_ptr(), q_indptr.data_ptr(), accepted_len.data_ptr(),
                               out.data_ptr(), status.data_ptr(), _stream(dev)))
    return out, status


def draft_confidence(draft_logits, draft_ids, q_indptr, vocab=None, want_token_conf=True, ws: Optional[Workspace] = None):
    """spx_draft_confidence on the current stream.  Returns (conf_max, conf_tok or None, req_conf, ws)."""
    _require_cuda(draft_logits, q_indptr)
    lib = load_library()
    dev = q_indptr.device
    B = q_indptr.numel() - 1
    TD = draft_logits.shape[0]
    a = ConfArgs()
    a.batch, a.total_q = B, TD + B
    a.vocab = int(vocab if vocab is not None else draft_logits.shape[1])
    a.logits_row_stride = draft_logits.stride(0) if TD else a.vocab + (-a.vocab) % 8
    a.logits_dtype = _dtype_code(draft_logits)
    conf_max = torch.empty(TD, dtype=torch.float32, device=dev)
    conf_tok = torch.empty(TD, dtype=torch.float32, device=dev) if want_token_conf and draft_ids is not None else None
    req_conf = torch.empty(B, dtype=torch.float32, device=dev)
    a.draft_logits, a.draft_token_ids, a.q_indptr = _ptr(draft_logits), _ptr(draft_ids), q_indptr.data_ptr()
    a.conf_max, a.conf_tok, a.req_conf = _ptr(conf_max), _ptr(conf_tok), _ptr(req_conf)
    need = int(lib.spx_draft_confidence_workspace(C.byref(a)))
    if need == 0:
        raise SpxError(ERR_INVALID_ARG, "invalid arguments for workspace sizing")
    if ws is None:
        ws = Workspace.allocate(need, dev)
    ws.ensure(need)
    _check(lib.spx_draft_confidence(C.byref(a), ws.buf.data_ptr(), ws.buf.numel(), ws.status.data_ptr(), _stream(dev)))
    return conf_max, conf_tok, req_conf, ws


def select_speculation(confidence, k_in, alpha: float, out: Optional[torch.Tensor] = None,
                       status: Optional[torch.Tensor] = None, n_drop: Optional[torch.Tensor] = None):
    """spx_select_speculation on the current stream.  Returns (k_out, n_drop [1] int32 on the device, status)."""
    _require_cuda(confidence, k_in)
    lib = load_library()
    dev = k_in.device
    if out is None:
        out = torch.empty_like(k_in)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    if n_drop is None:
        n_drop = torch.zeros(1, dtype=torch.int32, device=dev)
    _check(lib.spx_select_speculation(k_in.numel(), _ptr(confidence), _ptr(k_in), float(alpha), _ptr(out),
                                      n_drop.data_ptr(), status.data_ptr(), _stream(dev)))
    return out, n_drop, status


def lookahead_memory(ell, tau, prec, pp: int, theta: float, horizon: int = 64):
    """spx_lookahead_memory on the current stream: [horizon] float64 on the device."""
    _require_cuda(ell, tau, prec)
    lib = load_library()
    out = torch.empty(horizon, dtype=torch.float64, device=ell.device)
    _check(lib.spx_lookahead_memory(ell.numel(), _ptr(ell), _ptr(tau), _ptr(prec), int(pp), float(theta), int(horizon),
                                    out.data_ptr(), _stream(ell.device)))
    return out


def sp_effective_batch(batch: float, stages: int, theta: float) -> float:
    return float(load_library().spx_sp_effective_batch(float(batch), int(stages), float(theta)))


def selective_batch(batch: float, stages: int, alpha: float) -> float:
    return float(load_library().spx_selective_batch(float(batch), int(stages), float(alpha)))


def selective_effective_batch(batch: float, stages: int, alpha: float, theta_alpha: float) -> float:
    return float(load_library().spx_selective_effective_batch(float(batch), int(stages), float(alpha), float(theta_alpha)))


def delay_gain(iterations: float, pdr: float, running: float, i_delay: float, i_wait) -> float:
    w = (C.c_double * len(i_wait))(*[float(x) for x in i_wait])
    return float(load_library().spx_delay_gain(float(iterations), len(i_wait), float(pdr), float(running), float(i_delay), w))


LM_TILE_COLS = 128


def lm_head(hidden, weight, logits: Optional[torch.Tensor] = None, want_stats: bool = True,
            tile_stats: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None):
    """spx_lm_head on the current stream.  Returns (logits [rows, stride] bf16, tile_stats or None, status)."""
    _require_cuda(hidden, weight)
    lib = load_library()
    dev = hidden.device
    rows, K = hidden.shape
    V = weight.shape[0]
    if logits is None:
        stride = V + (-V) % 8
        logits = torch.empty((rows, stride), dtype=torch.bfloat16, device=dev)
    if want_stats and tile_stats is None:
        tile_stats = torch.empty((rows, (V + LM_TILE_COLS - 1) // LM_TILE_COLS, 2), dtype=torch.float32, device=dev)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    a = LmHeadArgs()
    a.rows, a.hidden_dim, a.vocab = rows, K, V
    a.hidden, a.weight, a.logits = _ptr(hidden), _ptr(weight), _ptr(logits)
    a.logits_row_stride = logits.stride(0)
    a.tile_stats = _ptr(tile_stats) if want_stats else None
    _check(lib.spx_lm_head(C.byref(a), status.data_ptr(), _stream(dev)))
    return logits, (tile_stats if want_stats else None), status
