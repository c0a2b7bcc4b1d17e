"""The sampling half without caller-provided scratch (spx_rejection_sample_static).

For users of the library who cannot allocate device memory where they call it - inside a stream
capture, under a runtime whose allocator owns the GPU, in a plugin that only receives its tensors -
the sampling half also exists with its scratch in a fixed array inside the library.  This file
checks, through the C ABI, that it returns exactly what spx_rejection_sample returns, on two calls
in a row with different batches (the array keeps the first call's contents, which must not
matter), and that a batch needing more scratch than the fixed array is refused with
SPX_ERR_WORKSPACE.  It is collected last so that a failure here cannot hide another test's result,
and it passes both alone in a fresh process and after the rest of the suite.
"""
import ctypes as C

import pytest
import torch

import spx_workloads as W
import paper_2609_34370_b200 as spx
from paper_2609_34370_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both_ways(b):
    ref_acc, ref_tok, _, ws = spx.rejection_sample(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr,
                                                   b.u_accept, b.u_sample)
    acc, tok, status = spx.rejection_sample_static(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr,
                                                   b.u_accept, b.u_sample)
    torch.cuda.synchronize()
    assert int(ws.status.item()) == 0 and int(status.item()) == 0
    # same kernels, same arithmetic: the tolerance of the sampling tests is bit-exactness
    assert torch.equal(acc, ref_acc)
    assert torch.equal(tok, ref_tok)
    return acc, tok


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row():
    first = W.generate(W.scaled(W.CONFIGS[1], batch=8, ctx_div=16, vocab=50000)).to(DEV)
    second = W.generate(W.scaled(W.CONFIGS[4], batch=20, ctx_div=32, vocab=128256)).to(DEV)
    acc1, tok1 = _both_ways(first)
    acc2, tok2 = _both_ways(second)          # the array still holds the first call's statistics
    acc1b, tok1b = _both_ways(first)         # and now the second call's
    assert torch.equal(acc1, acc1b) and torch.equal(tok1, tok1b)
    assert acc2.numel() == 20


def test_static_scratch_refuses_batches_beyond_its_fixed_size():
    lib = spx.load_library()
    s = binding.SampleArgs()
    s.batch, s.vocab, s.logits_row_stride, s.logits_dtype = 1024, 128256, 128256, binding.BF16
    s.total_q = s.batch * 16                   # 31 744 logits rows: about 16 MB of scratch
    fake = 0x1000                              # never dereferenced: the size check comes first
    for name in ("target_logits", "draft_logits", "draft_token_ids", "q_indptr", "u_accept", "u_sample",
                 "accepted_len", "out_tokens"):
        setattr(s, name, fake)
    assert lib.spx_workspace_size(None, C.byref(s)) > spx.STATIC_SCRATCH_BYTES
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    code = lib.spx_rejection_sample_static(C.byref(s), status.data_ptr(), None)
    assert code == binding.ERR_WORKSPACE
    assert b"workspace" in lib.spx_status_string(code)
