"""The C-ABI library loads without a GPU, exports what include/spx.h declares, and rejects bad
host-visible arguments before touching the device (CPU only: no kernel is launched here)."""
import ctypes as C
import os
import re

import pytest

import paper_2609_34370_b200 as spx
from paper_2609_34370_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return spx.load_library()


def test_header_and_exports_agree(lib):
    header = open(os.path.join(ROOT, "include", "spx.h")).read()
    declared = set(re.findall(r"\b(spx_[a-z_]+)\s*\(", header))
    assert declared == set(spx.exported_symbols())
    for name in declared:
        assert hasattr(lib, name), name


def _attn(**over):
    a = binding.AttnArgs()
    a.batch, a.total_q, a.max_q_len = 4, 20, 5
    a.num_q_heads, a.num_kv_heads, a.head_dim, a.page_size = 8, 2, 64, 16
    a.num_pages, a.max_pages_per_req, a.kv_dtype, a.sm_scale = 40, 17, binding.F32, 0.0
    a.kv_stride_page, a.kv_stride_head, a.kv_stride_token = 2 * 16 * 64, 16 * 64, 64
    for k, v in over.items():
        setattr(a, k, v)
    return a


def _sample(**over):
    s = binding.SampleArgs()
    s.batch, s.total_q, s.vocab, s.logits_row_stride, s.logits_dtype = 4, 20, 1024, 1024, binding.F32
    for k, v in over.items():
        setattr(s, k, v)
    return s


def test_workspace_size_is_positive_and_monotone(lib):
    a, s = _attn(), _sample()
    wa = lib.spx_workspace_size(C.byref(a), None)
    ws_ = lib.spx_workspace_size(None, C.byref(s))
    both = lib.spx_workspace_size(C.byref(a), C.byref(s))
    assert wa > 0 and ws_ > 0 and both == wa + ws_ and both % 256 == 0
    bigger = lib.spx_workspace_size(C.byref(_attn(batch=8, total_q=40)), None)
    assert bigger > wa


@pytest.mark.parametrize("over", [dict(head_dim=96), dict(num_q_heads=7), dict(page_size=24),
                                  dict(max_q_len=17), dict(num_q_heads=64, num_kv_heads=2, max_q_len=8)])
def test_unsupported_shapes_are_refused(lib, over):
    a = _attn(**over)
    assert lib.spx_workspace_size(C.byref(a), None) == 0
    status = C.c_int32(0)
    code = lib.spx_verify_attention(C.byref(a), None, 0, C.byref(status), None)
    assert code == binding.ERR_UNSUPPORTED


@pytest.mark.parametrize("over", [dict(batch=-1), dict(total_q=2), dict(kv_dtype=7), dict(kv_stride_token=8),
                                  dict(sm_scale=-1.0)])
def test_invalid_attention_arguments(lib, over):
    a = _attn(**over)
    status = C.c_int32(0)
    assert lib.spx_verify_attention(C.byref(a), None, 0, C.byref(status), None) == binding.ERR_INVALID_ARG


def test_null_pointers_and_workspace_are_refused_before_any_launch(lib):
    status = C.c_int32(0)
    a = _attn()                                  # all data pointers NULL
    assert lib.spx_verify_attention(C.byref(a), None, 0, C.byref(status), None) == binding.ERR_INVALID_ARG
    s = _sample()
    assert lib.spx_rejection_sample(C.byref(s), None, 0, C.byref(status), None) == binding.ERR_INVALID_ARG
    assert lib.spx_rejection_sample(C.byref(_sample(logits_row_stride=1023)), None, 0, C.byref(status), None) \
        == binding.ERR_INVALID_ARG
    assert lib.spx_rejection_sample(C.byref(_sample(vocab=0)), None, 0, C.byref(status), None) \
        == binding.ERR_INVALID_ARG
    # pointers present (fake, never dereferenced on the host) but no workspace
    fake = 0x1000
    s2 = _sample(target_logits=fake, draft_logits=fake, draft_token_ids=fake, q_indptr=fake, u_accept=fake,
                 u_sample=fake, accepted_len=fake, out_tokens=fake)
    assert lib.spx_rejection_sample(C.byref(s2), None, 0, C.byref(status), None) == binding.ERR_WORKSPACE
    assert lib.spx_rejection_sample(C.byref(s2), C.c_void_p(0x1001), 1 << 30, C.byref(status), None) \
        == binding.ERR_WORKSPACE
    assert lib.spx_rejection_sample(C.byref(s2), C.c_void_p(0x1000), 1 << 30, None, None) == binding.ERR_INVALID_ARG


def test_status_strings(lib):
    assert lib.spx_status_string(0) == b"ok"
    assert b"workspace" in lib.spx_status_string(3)


def test_binding_refuses_host_tensors():
    import torch
    t = torch.zeros(2, 8)
    with pytest.raises(spx.SpxError):
        spx.rejection_sample(t, t[:0], torch.zeros(0, dtype=torch.int32), torch.tensor([0, 1, 2], dtype=torch.int32),
                             torch.zeros(0), torch.zeros(2))


def test_calls_around_the_step_refuse_bad_arguments_before_any_launch(lib):
    status = C.c_int32(0)
    fake = C.c_void_p(0x1000)                                       # never dereferenced: every call below fails validation first
    # KV append / rollback
    ka = binding.KvAppendArgs()
    assert lib.spx_kv_append(None, C.byref(status), None) == binding.ERR_INVALID_ARG
    ka.batch, ka.total_q, ka.num_kv_heads, ka.head_dim, ka.page_size, ka.num_pages, ka.max_pages_per_req = 2, 6, 8, 128, 12, 10, 4
    ka.kv_dtype, ka.kv_stride_page, ka.kv_stride_head, ka.kv_stride_token = 0, 8 * 12 * 128, 12 * 128, 128
    assert lib.spx_kv_append(C.byref(ka), C.byref(status), None) == binding.ERR_UNSUPPORTED      # page size not a power of two
    ka.page_size = 16
    assert lib.spx_kv_append(C.byref(ka), C.byref(status), None) == binding.ERR_INVALID_ARG      # null pointers
    assert lib.spx_kv_append(C.byref(ka), None, None) == binding.ERR_INVALID_ARG
    assert lib.spx_kv_rollback(-1, fake, fake, fake, fake, C.byref(status), None) == binding.ERR_INVALID_ARG
    assert lib.spx_kv_rollback(3, None, fake, fake, fake, C.byref(status), None) == binding.ERR_INVALID_ARG
    assert lib.spx_kv_rollback(0, None, None, None, None, C.byref(status), None) == binding.OK   # empty batch: nothing to do
    # selection
    for alpha in (-0.1, 1.5, float("nan")):
        assert lib.spx_select_speculation(4, fake, fake, alpha, fake, None, C.byref(status), None) == binding.ERR_INVALID_ARG
    assert lib.spx_select_speculation(4, None, fake, 0.3, fake, None, C.byref(status), None) == binding.ERR_INVALID_ARG
    # confidence
    ca = binding.ConfArgs()
    ca.batch, ca.total_q, ca.vocab, ca.logits_row_stride, ca.logits_dtype = 4, 12, 1000, 1001, 0
    assert lib.spx_draft_confidence_workspace(C.byref(ca)) == 0                                  # stride not a multiple of 8
    ca.logits_row_stride = 1000
    assert lib.spx_draft_confidence_workspace(C.byref(ca)) > 0
    assert lib.spx_draft_confidence(C.byref(ca), None, 0, C.byref(status), None) == binding.ERR_INVALID_ARG
    # look-ahead memory
    for pp, theta, horizon in ((0, 0.5, 64), (2, -0.1, 64), (2, 0.5, 0), (2, 0.5, 257)):
        assert lib.spx_lookahead_memory(4, fake, fake, fake, pp, theta, horizon, fake, None) == binding.ERR_INVALID_ARG
    assert lib.spx_lookahead_memory(4, None, fake, fake, 2, 0.5, 64, fake, None) == binding.ERR_INVALID_ARG
    # LM head
    la = binding.LmHeadArgs()
    la.rows, la.hidden_dim, la.vocab, la.logits_row_stride = 4, 60, 100, 104
    assert lib.spx_lm_head(C.byref(la), C.byref(status), None) == binding.ERR_UNSUPPORTED        # hidden size not a multiple of 8
    la.hidden_dim = 64
    assert lib.spx_lm_head(C.byref(la), C.byref(status), None) == binding.ERR_INVALID_ARG        # null pointers
    la.logits_row_stride = 96
    assert lib.spx_lm_head(C.byref(la), C.byref(status), None) == binding.ERR_INVALID_ARG        # stride below the vocabulary
    assert status.value == 0


def test_timeline_is_a_build_option():
    """The regular build records no per-CTA stamps: the call reports its dimensions and refuses."""
    import ctypes as C
    lib = spx.load_library()
    nk, nc = C.c_int32(0), C.c_int32(0)
    st = lib.spx_debug_timeline(None, 0, C.byref(nk), C.byref(nc))
    assert st == binding.ERR_UNSUPPORTED and nk.value >= 7 and nc.value >= 148
