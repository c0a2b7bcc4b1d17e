"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Small cases and the full-size workloads alike are compared element by element on every request.
Tolerances are in tests/parity_util.py; every buffer the library writes sits between guard bands
that are checked after the call (tests/conftest.py, parity_util.Guarded).
"""
import dataclasses

import pytest
import torch

import oracle
import spx_workloads as W
import paper_2609_34370_b200 as spx
from parity_util import (check_attention, check_sampling, gpu_attention, gpu_sample, oracle_attention)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _small_specs():
    c = W.CONFIGS
    return [
        c[0],
        W.scaled(c[1], batch=6, ctx_div=4, vocab=20000),       # several 128-token tiles + ragged tails
        W.scaled(c[2], batch=8, ctx_div=4, vocab=9000),
        W.scaled(c[3], batch=2, ctx_div=8, vocab=32000),       # 4096 tokens, page 32, k = 8 (36 packed rows)
        W.scaled(c[4], batch=12, ctx_div=8, vocab=128256),     # ragged k incl. 0, fragmented pool
    ]


@pytest.mark.parametrize("idx", range(5))
@pytest.mark.parametrize("layout", ["HND", "NHD"])
def test_small_workloads_match_oracle(idx, layout):
    spec = _small_specs()[idx]
    if layout == "NHD" and idx in (2, 3):
        pytest.skip("strided layout covered by the other workloads")
    b_cpu = W.generate(spec, layout=layout)
    b = b_cpu.to(DEV)
    out, lse, ws = gpu_attention(b)
    assert int(ws.status.item()) == 0
    ref_o, ref_l = oracle_attention(b_cpu)
    check_attention(b_cpu, out, lse, ref_o, ref_l)
    acc, tok, ratio, ws2 = gpu_sample(b, want_ratio=True)
    assert int(ws2.status.item()) == 0
    rep = check_sampling(b_cpu, acc, tok)
    assert not rep.hard_mismatch, rep
    assert rep.exact + rep.accept_near_tie + rep.cdf_near_tie == rep.requests
    # the diagnostic ratio is p/q of every consulted draft
    ref = oracle.rejection_sample(b_cpu.target_logits, b_cpu.draft_logits, b_cpu.draft_ids, b_cpu.q_indptr,
                                  b_cpu.u_accept, b_cpu.u_sample)
    consulted = ~torch.isnan(ref.rho)
    got = ratio.cpu().double()
    assert torch.equal(torch.isnan(got), ~consulted) or rep.accept_near_tie > 0
    both = consulted & ~torch.isnan(got)
    assert torch.allclose(got[both], ref.rho[both], rtol=2e-5)


def test_attention_plan_large_batch_and_long_requests():
    """The work plan cuts the concatenated tile axis of all (request, kv head) pairs into one range
    per CTA.  A batch above 1024 requests takes the planner's multi-pass path (prefix sums in
    global memory, many whole pairs per range); a batch of few long requests makes every pair
    span several ranges (several partial chunks per pair)."""
    many = dataclasses.replace(W.CONFIGS[1], batch=1100, vocab=64, ctx=("uniform", 20, 400),
                               k=("choice", (0, 1, 2, 4)), name="many-short")
    few = dataclasses.replace(W.CONFIGS[1], batch=3, vocab=64, ctx=("uniform", 9000, 14000),
                              k=("const", 4), name="few-long")
    for spec, sample in ((many, 40), (few, None)):
        b_cpu = W.generate(spec)
        b = b_cpu.to(DEV)
        out, lse, ws = gpu_attention(b)
        assert int(ws.status.item()) == 0
        reqs = list(range(b_cpu.batch)) if sample is None else list(range(0, b_cpu.batch, b_cpu.batch // sample))
        ref_o, ref_l = oracle_attention(b_cpu, reqs)
        check_attention(b_cpu, out, lse, ref_o, ref_l, reqs)
        assert not torch.isnan(out.float()).any()


def test_bf16_variant_of_tiny_workload():
    import dataclasses
    spec = dataclasses.replace(W.CONFIGS[0], dtype="bf16", name="tiny-bf16")
    b_cpu = W.generate(spec)
    b = b_cpu.to(DEV)
    out, lse, _ = gpu_attention(b)
    ref_o, ref_l = oracle_attention(b_cpu)
    check_attention(b_cpu, out, lse, ref_o, ref_l)
    acc, tok, _, _ = gpu_sample(b)
    assert not check_sampling(b_cpu, acc, tok).hard_mismatch


def test_verify_step_equals_the_two_halves_and_is_deterministic():
    from paper_2609_34370_b200 import binding
    spec = W.scaled(W.CONFIGS[4], batch=10, ctx_div=8, vocab=40000)
    b = W.generate(spec).to(DEV)
    s = spec
    out_a, lse_a, _ = gpu_attention(b, max_q_len=7)
    acc_a, tok_a, _, _ = gpu_sample(b)
    results = []
    for _ in range(2):
        out = torch.empty_like(b.q)
        lse = torch.empty(b.q.shape[:2], dtype=torch.float32, device=DEV)
        acc = torch.empty(b.batch, dtype=torch.int32, device=DEV)
        tok = torch.empty(b.total_q, dtype=torch.int32, device=DEV)
        a = binding.make_attn_args(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                                   s.num_kv_heads, s.page_size, b.num_pages, out, lse, max_q_len=7)
        sa = binding.make_sample_args(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept,
                                      b.u_sample, acc, tok)
        ws = spx.Workspace.allocate(spx.workspace_size(a, sa), DEV)
        ws.buf.fill_(0xA5)                         # stale workspace contents must not matter
        spx.verify_step(a, sa, ws, DEV)
        torch.cuda.synchronize()
        assert int(ws.status.item()) == 0
        assert spx.last_launch_count() >= 5
        results.append((out, lse, acc, tok))
    for out, lse, acc, tok in results:
        assert torch.equal(out, out_a) and torch.equal(lse, lse_a)
        assert torch.equal(acc, acc_a) and torch.equal(tok, tok_a)


def test_verify_step_can_be_captured_in_a_cuda_graph():
    """The step only enqueues work (its internal stream is forked from and joined to the caller's
    stream by events), so a stream capture of one call replays it: same outputs, bit for bit."""
    from paper_2609_34370_b200 import binding
    spec = W.scaled(W.CONFIGS[1], batch=12, ctx_div=4, vocab=50000)
    b = W.generate(spec).to(DEV)
    out = torch.empty_like(b.q)
    lse = torch.empty(b.q.shape[:2], dtype=torch.float32, device=DEV)
    acc = torch.empty(b.batch, dtype=torch.int32, device=DEV)
    tok = torch.empty(b.total_q, dtype=torch.int32, device=DEV)
    a = binding.make_attn_args(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                               spec.num_kv_heads, spec.page_size, b.num_pages, out, lse)
    sa = binding.make_sample_args(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample,
                                  acc, tok)
    ws = spx.Workspace.allocate(spx.workspace_size(a, sa), DEV)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for _ in range(3):                         # warm-up outside the capture (function attributes, side stream)
            spx.verify_step(a, sa, ws, DEV)
    torch.cuda.synchronize()
    want = (out.clone(), lse.clone(), acc.clone(), tok.clone())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        spx.verify_step(a, sa, ws, DEV)
    torch.cuda.synchronize()
    for t in (out, lse, acc, tok):
        t.zero_()
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    assert int(ws.status.item()) == 0
    for got, ref in zip((out, lse, acc, tok), want):
        assert torch.equal(got, ref)


def test_edge_cases_k0_minimal_context_and_page_boundaries():
    # hand-made lengths: L = k+1 (no prior context), L exactly on page/tile boundaries, k = 0, k = 15
    import dataclasses
    base = dataclasses.replace(W.CONFIGS[1], batch=1, vocab=777, name="edge")
    cases = [(1, 0), (6, 5), (16, 15), (128, 3), (129, 3), (127, 0), (256, 7), (257, 1), (2048, 15), (16, 0)]
    for L, k in cases:
        spec = dataclasses.replace(base, ctx=("const", L), k=("const", k))
        b_cpu = W.generate(spec, seed=1000 + L * 16 + k)
        # vocab 777 is not a multiple of the 16-byte vector: rows are padded to a stride of 784
        padded = {}
        for name in ("target_logits", "draft_logits"):
            t = getattr(b_cpu, name)
            padded[name] = torch.full((t.shape[0], 784), 30.0, dtype=t.dtype)      # poison in the padding
            padded[name][:, :777] = t
            setattr(b_cpu, name, padded[name][:, :777])
        b = b_cpu.to(DEV)
        b.target_logits = padded["target_logits"].to(DEV)[:, :777]
        b.draft_logits = padded["draft_logits"].to(DEV)[:, :777]
        out, lse, ws = gpu_attention(b)
        assert int(ws.status.item()) == 0
        ref_o, ref_l = oracle_attention(b_cpu)
        check_attention(b_cpu, out, lse, ref_o, ref_l)
        acc, tok, _, _ = gpu_sample(b)
        assert not check_sampling(b_cpu, acc, tok).hard_mismatch, (L, k)


def test_empty_batch_is_a_no_op():
    from paper_2609_34370_b200 import binding
    import ctypes as C
    lib = spx.load_library()
    a = binding.AttnArgs()
    a.batch, a.total_q, a.num_q_heads, a.num_kv_heads, a.head_dim, a.page_size = 0, 0, 8, 2, 64, 16
    a.kv_stride_page, a.kv_stride_head, a.kv_stride_token = 2048, 1024, 64
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    s = binding.SampleArgs()
    s.batch, s.total_q, s.vocab, s.logits_row_stride, s.logits_dtype = 0, 0, 64, 64, 1
    ws = torch.empty(spx.workspace_size(a, s), dtype=torch.uint8, device=DEV)
    assert lib.spx_verify_attention(C.byref(a), ws.data_ptr(), ws.numel(), st.data_ptr(), None) == 0
    assert lib.spx_rejection_sample(C.byref(s), ws.data_ptr(), ws.numel(), st.data_ptr(), None) == 0
    torch.cuda.synchronize()
    assert int(st.item()) == 0


def test_needle_at_mask_edge_and_page_edges_on_gpu():
    import dataclasses
    spec = dataclasses.replace(W.CONFIGS[1], batch=1, vocab=64, ctx=("const", 1000), k=("const", 5), name="needle")
    b_cpu = W.generate(spec)
    L, k, P = 1000, 5, spec.page_size
    G = spec.num_q_heads // spec.num_kv_heads
    for t_needle in (0, 15, 16, 127, 128, 993, 994, 997, 999):
        bb = b_cpu.clone()
        j, h = 2, 9                                                  # query position 2, q-head 9 -> kv-head 2
        qv = bb.q[j, h].float()
        page = int(bb.block_table[0, t_needle // P])
        bb.k_cache[page, h // G, t_needle % P, :] = (60.0 * qv / qv.norm()).to(bb.k_cache.dtype)
        out, lse, _ = gpu_attention(bb.to(DEV))
        visible = t_needle <= L - (k + 1) + j
        hit = torch.allclose(out[j, h].float().cpu(), bb.v_cache[page, h // G, t_needle % P].float(), atol=3e-2)
        assert hit == visible, t_needle
        ref_o, ref_l = oracle_attention(bb)
        check_attention(bb, out, lse, ref_o, ref_l)


def test_device_side_faults_are_reported_not_fatal():
    spec = W.scaled(W.CONFIGS[1], batch=4, ctx_div=8, vocab=5000)
    b_cpu = W.generate(spec)
    ref_o, ref_l = oracle_attention(b_cpu)
    ref = oracle.rejection_sample(b_cpu.target_logits, b_cpu.draft_logits, b_cpu.draft_ids, b_cpu.q_indptr,
                                  b_cpu.u_accept, b_cpu.u_sample)
    # bad sequence length for request 1 -> BAD_LEN, zero rows, other requests untouched
    bad = b_cpu.clone()
    bad.seq_lens[1] = 3
    out, lse, ws = gpu_attention(bad.to(DEV))
    assert int(ws.status.item()) & spx.DEV_BAD_LEN
    check_attention(b_cpu, out, lse, ref_o, ref_l, reqs=[0, 2, 3])
    q0, q1 = int(b_cpu.q_indptr[1]), int(b_cpu.q_indptr[2])
    assert (out[q0:q1] == 0).all() and torch.isnan(lse[q0:q1]).all()
    # page id out of range for request 2 -> BAD_PAGE, kernel completes
    bad = b_cpu.clone()
    bad.block_table[2, 1] = b_cpu.num_pages + 5
    out, lse, ws = gpu_attention(bad.to(DEV))
    assert int(ws.status.item()) & spx.DEV_BAD_PAGE
    check_attention(b_cpu, out, lse, ref_o, ref_l, reqs=[0, 1, 3])
    q0, q1 = int(b_cpu.q_indptr[2]), int(b_cpu.q_indptr[3])
    assert (out[q0:q1] == 0).all() and torch.isnan(lse[q0:q1]).all()      # sentinel rows, split pair or not
    # draft id out of range for request 0 -> BAD_TOKEN, that request emits n = 0 and -1s
    bad = b_cpu.clone()
    bad.draft_ids[0] = spec.vocab
    acc, tok, _, ws = gpu_sample(bad.to(DEV))
    assert int(ws.status.item()) & spx.DEV_BAD_TOKEN
    q1 = int(b_cpu.q_indptr[1])
    assert int(acc[0]) == 0 and (tok[:q1] == -1).all()
    assert torch.equal(acc[1:].cpu(), ref.accepted_len[1:]) and torch.equal(tok[q1:].cpu(), ref.out_tokens[q1:])


def test_vocabulary_beyond_the_staged_segment_masses():
    """A vocabulary of more than 128 segments of 8192 tokens: the draw reads the segment masses
    beyond its shared-memory staging array in place.  Three requests: one rejected early (the
    residual draw lands in a late segment for u_sample near 1), one bonus draw, one k = 0."""
    V = 8192 * 130 + 40
    g = torch.Generator().manual_seed(11)
    T = (torch.randn(5, V, generator=g) * 2).to(torch.bfloat16)
    qi = torch.tensor([0, 2, 4, 5], dtype=torch.int32)                  # k = 1, 1, 0
    Dr = torch.stack([T[0].roll(7), T[2]]).clone()                      # request 0: another law; request 1: q == p
    ids = torch.tensor([int(torch.argmax(Dr[0].float())), 123], dtype=torch.int32)
    ua = torch.tensor([0.999999, 0.5])
    for us_val in (0.003, 0.5, 1 - 2.0 ** -20):
        us = torch.full((3,), us_val)
        ref = oracle.rejection_sample(T, Dr, ids, qi, ua, us)
        acc, tok, _, ws = spx.rejection_sample(T.to(DEV), Dr.to(DEV), ids.to(DEV), qi.to(DEV), ua.to(DEV), us.to(DEV))
        torch.cuda.synchronize()
        assert int(ws.status.item()) == 0
        assert ref.accepted_len.tolist() == [0, 1, 0]
        assert torch.equal(acc.cpu(), ref.accepted_len)
        b = type("B", (), {})()
        b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample = T, Dr, ids, qi, ua, us
        b.batch = 3
        b.spec = type("S", (), {"vocab": V})
        rep = check_sampling(b, acc, tok, ref)
        assert not rep.hard_mismatch, rep


def test_sampler_special_cases_on_gpu():
    # q == p accepts everything; disjoint supports reject at 0; k = 0 plain sampling; u_sample extremes
    V = 9000
    g = torch.Generator().manual_seed(4)
    T = (torch.randn(12, V, generator=g) * 3).to(torch.bfloat16)
    qi = torch.tensor([0, 4, 8, 9, 12], dtype=torch.int32)            # k = 3, 3, 0, 2
    Dr = torch.stack([T[0], T[1], T[2], T[4], T[5], T[6], T[9], T[10]]).clone()
    Dr[3:6] = -1e4
    Dr[3:6, 5000:] = 0.0                                             # request 1: draft mass where target is ~0
    Tm = T.clone()
    Tm[4:8, 5000:] = -1e4
    ids = torch.tensor([5, 6, 7, 6000, 6001, 6002, 11, 12], dtype=torch.int32)
    ua = torch.tensor([0.999, 0.5, 0.0, 0.0, 0.0, 0.0, 0.9999, 0.3])
    for us_val in (0.0, 0.37, 1 - 2.0 ** -24):
        us = torch.full((4,), us_val)
        ref = oracle.rejection_sample(Tm, Dr, ids, qi, ua, us)
        acc, tok, _, ws = spx.rejection_sample(Tm.to(DEV), Dr.to(DEV), ids.to(DEV), qi.to(DEV), ua.to(DEV),
                                               us.to(DEV))
        torch.cuda.synchronize()
        assert ref.accepted_len.tolist() == [3, 0, 0, 2]
        assert acc.cpu().tolist() == [3, 0, 0, 2]

        class _B:
            pass
        bb = _B()
        bb.batch, bb.q_indptr, bb.u_accept, bb.u_sample = 4, qi, ua, us
        bb.target_logits, bb.draft_logits, bb.draft_ids = Tm, Dr, ids
        bb.spec = type("S", (), {"vocab": V})
        rep = check_sampling(bb, acc, tok, ref)
        assert not rep.hard_mismatch, (us_val, rep, tok.cpu().tolist(), ref.out_tokens.tolist())


@pytest.mark.parametrize("idx", [1, 2, 3, 4])
def test_full_size_workloads(idx):
    """The benchmark's sizes and launch configuration: attention and sampler compared with the oracle
    on every request (the float64 oracle does a whole workload in seconds on the host cores)."""
    spec = W.CONFIGS[idx]
    b = W.generate(spec, device=DEV)
    out, lse, ws = gpu_attention(b, max_q_len=max(b.k_host) + 1)
    assert int(ws.status.item()) == 0
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
    # the work split depends only on the lengths, so repeated launches must agree bit for bit (a
    # race between the kernel's roles would show up here)
    for _ in range(3):
        out2, lse2, _ = gpu_attention(b, ws=ws, max_q_len=max(b.k_host) + 1)
        assert torch.equal(out, out2) and torch.equal(lse, lse2)
    b_cpu = b.to("cpu")
    ref_o, ref_l = oracle_attention(b_cpu)
    check_attention(b_cpu, out, lse, ref_o, ref_l)
    # per request as well: the batch-wide relative RMS must not hide one bad short request
    for r in range(b_cpu.batch):
        rows = slice(int(b_cpu.q_indptr[r]), int(b_cpu.q_indptr[r + 1]))
        d = out[rows].cpu().double() - ref_o[rows]
        assert float(d.norm() / ref_o[rows].norm()) <= 1e-2, r
    acc, tok, _, ws2 = gpu_sample(b)
    assert int(ws2.status.item()) == 0
    rep = check_sampling(b_cpu, acc, tok)
    assert not rep.hard_mismatch, rep
    print(f"\n[{spec.name}] sampling: exact {rep.exact}/{rep.requests}, accept-near-tie {rep.accept_near_tie}, "
          f"cdf-near-tie {rep.cdf_near_tie}, accept-band-eligible drafts {rep.accept_band_eligible}")


def test_a_lost_page_at_long_context_fails_the_gates():
    """At 32768 tokens of context one page of 32 tokens carries 1e-3 of a row's weight: the output
    moves by less than the contract's 2e-2, so the LSE gate has to catch it.  The kernel runs on a
    batch whose block table skips one middle page (a legitimate input: the same request, 32 tokens
    shorter) and is held against the oracle's result for the full request."""
    spec = dataclasses.replace(W.CONFIGS[3], batch=1, vocab=64, name="lost-page")
    b_cpu = W.generate(spec)
    ref_o, ref_l = oracle_attention(b_cpu)
    out, lse, _ = gpu_attention(b_cpu.to(DEV))
    check_attention(b_cpu, out, lse, ref_o, ref_l)                       # the full request passes
    lost = b_cpu.clone()
    npages = int(lost.seq_lens[0]) // spec.page_size
    drop = npages // 2
    lost.block_table[0, drop:npages - 1] = b_cpu.block_table[0, drop + 1:npages]
    lost.seq_lens[0] -= spec.page_size
    out2, lse2, ws = gpu_attention(lost.to(DEV))
    assert int(ws.status.item()) == 0
    assert float((out2.cpu().double() - ref_o).abs().max()) < 2e-2       # the contract bound alone is blind to it
    with pytest.raises(AssertionError):
        check_attention(b_cpu, out2, lse2, ref_o, ref_l)
