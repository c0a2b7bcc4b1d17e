"""Pins for the oracle's attention half (CPU only).

The oracle is checked against things other than itself: a library routine
(torch.nn.functional.scaled_dot_product_attention in float64 on the un-paged tensors), hand
worked closed forms, and invariants of the definition (weights sum to one, causality, page
placement, GQA head duplication).  Each test is chosen so that one plausible mistake - a wrong
page/slot index, an off-by-one in the causal limit, a wrong head group, a missing scale, a
transposed operand - fails it.
"""
import math

import pytest
import torch

import oracle
import spx_workloads as W


def _densify(b, r):
    """Un-page request r: K, V as [L, Hkv, D] float64 (index arithmetic only)."""
    s = b.spec
    L = b.seq_lens_host[r]
    P = s.page_size
    t = torch.arange(L)
    pages = b.block_table[r, (t // P).long()].long()
    slots = (t % P).long()
    if b.layout == "HND":
        K = b.k_cache[pages, :, slots, :]
        V = b.v_cache[pages, :, slots, :]
    else:
        K = b.k_cache[pages, slots, :, :]
        V = b.v_cache[pages, slots, :, :]
    return K.double(), V.double()


def _oracle(b, **kw):
    s = b.spec
    return oracle.verify_attention(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens,
                                   b.q_indptr, s.num_kv_heads, s.page_size, b.num_pages, **kw)


def _library_attention(b, r):
    """scaled_dot_product_attention (float64) with an explicit causal mask for request r."""
    s = b.spec
    K, V = _densify(b, r)                                   # [L, Hkv, D]
    L = K.shape[0]
    m = b.k_host[r] + 1
    q0 = int(b.q_indptr[r])
    Q = b.q[q0:q0 + m].double()                             # [m, Hq, D]
    G = s.num_q_heads // s.num_kv_heads
    Kh = K.permute(1, 0, 2).repeat_interleave(G, dim=0)     # [Hq, L, D]
    Vh = V.permute(1, 0, 2).repeat_interleave(G, dim=0)
    Qh = Q.permute(1, 0, 2)                                 # [Hq, m, D]
    pos = (L - m) + torch.arange(m)
    mask = torch.arange(L)[None, :] <= pos[:, None]         # [m, L]
    out = torch.nn.functional.scaled_dot_product_attention(Qh, Kh, Vh, attn_mask=mask)
    scores = (Qh @ Kh.transpose(1, 2)) / math.sqrt(s.head_dim)
    lse = torch.logsumexp(scores.masked_fill(~mask, -float("inf")), dim=-1)
    return out.permute(1, 0, 2), lse.permute(1, 0)          # [m, Hq, D], [m, Hq]


@pytest.mark.parametrize("layout", ["HND", "NHD"])
@pytest.mark.parametrize("cfg", [0, 4])
def test_matches_library_attention(cfg, layout):
    spec = W.CONFIGS[cfg]
    if cfg != 0:
        spec = W.scaled(spec, batch=6, ctx_div=32, vocab=64)
    b = W.generate(spec, layout=layout)
    out, lse = _oracle(b)
    for r in range(b.batch):
        ref_o, ref_l = _library_attention(b, r)
        q0 = int(b.q_indptr[r])
        m = b.k_host[r] + 1
        assert torch.allclose(out[q0:q0 + m], ref_o, rtol=1e-10, atol=1e-12)
        assert torch.allclose(lse[q0:q0 + m], ref_l, rtol=1e-10, atol=1e-12)


def _single_request(L, k, Hq, Hkv, D, P, dtype=torch.float32, seed=0):
    """A hand-built one-request batch with an identity page table (test-local helper)."""
    g = torch.Generator().manual_seed(seed)
    n_pages = (L + P - 1) // P
    spec = W.WorkloadSpec("hand", 99, 1, Hq, Hkv, D, P, 8, "fp32" if dtype == torch.float32 else "bf16",
                          ("const", L), ("const", k))
    kc = torch.randn(n_pages, Hkv, P, D, generator=g).to(dtype)
    vc = torch.randn(n_pages, Hkv, P, D, generator=g).to(dtype)
    q = torch.randn(k + 1, Hq, D, generator=g).to(dtype)
    bt = torch.arange(n_pages, dtype=torch.int32)[None, :]
    return W.VerifyBatch(spec=spec, layout="HND", num_pages=n_pages, q=q, k_cache=kc, v_cache=vc,
                         kv_strides=(Hkv * P * D, P * D, D), block_table=bt,
                         seq_lens=torch.tensor([L], dtype=torch.int32),
                         q_indptr=torch.tensor([0, k + 1], dtype=torch.int32),
                         target_logits=torch.zeros(k + 1, 8), draft_logits=torch.zeros(k, 8),
                         draft_ids=torch.zeros(k, dtype=torch.int32), u_accept=torch.zeros(k),
                         u_sample=torch.zeros(1), seq_lens_host=[L], k_host=[k])


def test_hand_worked_example():
    # D=1, scale forced to 1, q=1, keys log(1), log(2), log(3) -> weights 1/6, 2/6, 3/6.
    b = _single_request(L=3, k=0, Hq=1, Hkv=1, D=1, P=2)
    keys = torch.tensor([math.log(1.0), math.log(2.0), math.log(3.0)], dtype=torch.float32)
    vals = torch.tensor([6.0, 12.0, 18.0])
    b.k_cache.view(-1)[:3] = keys
    b.v_cache.view(-1)[:3] = vals
    b.q.fill_(1.0)
    out, lse = _oracle(b, sm_scale=1.0)
    w = torch.exp(keys.double())
    expect = float((w * vals.double()).sum() / w.sum())     # = 14 up to fp32 rounding of the logs
    assert abs(float(out[0, 0, 0]) - expect) < 1e-12
    assert abs(expect - 14.0) < 1e-5
    assert abs(float(lse[0, 0]) - math.log(float(w.sum()))) < 1e-12
    assert abs(float(lse[0, 0]) - math.log(6.0)) < 1e-6


def test_default_scale_is_inverse_sqrt_d():
    b = _single_request(L=9, k=1, Hq=2, Hkv=1, D=16, P=4)
    o0, l0 = _oracle(b)
    o1, l1 = _oracle(b, sm_scale=0.25)
    assert torch.equal(o0, o1) and torch.equal(l0, l1)
    o2, _ = _oracle(b, sm_scale=0.5)
    assert not torch.allclose(o0, o2)


def test_zero_keys_give_prefix_mean_and_log_count():
    L, k = 37, 3
    b = _single_request(L=L, k=k, Hq=4, Hkv=2, D=8, P=8)
    b.k_cache.zero_()
    out, lse = _oracle(b)
    K, V = _densify(b, 0)
    for j in range(k + 1):
        n_vis = L - (k + 1) + j + 1
        for h in range(4):
            mean = V[:n_vis, h // 2, :].mean(dim=0)
            assert torch.allclose(out[j, h], mean, rtol=1e-12, atol=1e-13)
            assert abs(float(lse[j, h]) - math.log(n_vis)) < 1e-12


def test_single_token_returns_its_value():
    b = _single_request(L=1, k=0, Hq=4, Hkv=2, D=8, P=4)
    out, lse = _oracle(b)
    for h in range(4):
        assert torch.equal(out[0, h], b.v_cache[0, h // 2, 0].double())


def test_weights_sum_to_one():
    # with V == 1 everywhere the output is the sum of the weights
    b = W.generate(W.CONFIGS[0])
    b.v_cache.fill_(1.0)
    out, _ = _oracle(b)
    assert torch.allclose(out, torch.ones_like(out), rtol=0, atol=1e-13)


def test_causal_mask_among_new_positions():
    b = W.generate(W.CONFIGS[0])
    out0, lse0 = _oracle(b)
    s = b.spec
    # perturb K/V at each request's LAST position: only query row k may change
    b2 = b.clone()
    for r, L in enumerate(b.seq_lens_host):
        t = L - 1
        page = int(b.block_table[r, t // s.page_size])
        b2.k_cache[page, :, t % s.page_size, :] += 3.0
        b2.v_cache[page, :, t % s.page_size, :] -= 5.0
    out1, lse1 = _oracle(b2)
    for r in range(b.batch):
        q0, k = int(b.q_indptr[r]), b.k_host[r]
        assert torch.equal(out0[q0:q0 + k], out1[q0:q0 + k])
        assert torch.equal(lse0[q0:q0 + k], lse1[q0:q0 + k])
        assert not torch.allclose(out0[q0 + k], out1[q0 + k])


def test_row_j_equals_plain_decode_of_truncated_context():
    b = W.generate(W.CONFIGS[0])
    out, lse = _oracle(b)
    for r in range(b.batch):
        q0, k, L = int(b.q_indptr[r]), b.k_host[r], b.seq_lens_host[r]
        for j in range(k + 1):
            o, l = oracle.verify_attention(
                b.q[q0 + j:q0 + j + 1], b.k_cache, b.v_cache, b.kv_strides, b.block_table[r:r + 1],
                torch.tensor([L - k + j], dtype=torch.int32), torch.tensor([0, 1], dtype=torch.int32),
                b.spec.num_kv_heads, b.spec.page_size, b.num_pages)
            assert torch.equal(o[0], out[q0 + j]) and torch.equal(l[0], lse[q0 + j])


def test_page_placement_invariance():
    b = W.generate(W.CONFIGS[0])
    out0, lse0 = _oracle(b)
    g = torch.Generator().manual_seed(5)
    perm = torch.randperm(b.num_pages, generator=g)
    b2 = b.clone()
    b2.k_cache[perm] = b.k_cache           # old page i moves to physical page perm[i]
    b2.v_cache[perm] = b.v_cache
    bt = b.block_table.clone()
    valid = bt >= 0
    bt[valid] = perm[bt[valid].long()].to(torch.int32)
    b2.block_table = bt
    out1, lse1 = _oracle(b2)
    assert torch.equal(out0, out1) and torch.equal(lse0, lse1)


def test_needle_key_selects_its_value():
    L, k, D, P = 70, 2, 16, 8
    for t_needle in (0, 7, 8, 63, 67, 68, 69):        # page edges and each of the last k+1 positions
        b = _single_request(L=L, k=k, Hq=2, Hkv=1, D=D, P=P, seed=t_needle)
        for j in range(k + 1):
            qv = b.q[j, 0].double()
            b2 = b.clone()
            b2.k_cache[t_needle // P, 0, t_needle % P, :] = (200.0 * qv / qv.norm()).float()
            out, _ = _oracle(b2)
            visible = t_needle <= L - (k + 1) + j
            hit = torch.allclose(out[j, 0], b2.v_cache[t_needle // P, 0, t_needle % P].double(), atol=1e-6)
            assert hit == visible, (t_needle, j)


def test_gqa_equals_duplicated_kv_heads():
    spec = W.scaled(W.CONFIGS[0], batch=3)
    b = W.generate(spec)
    out0, lse0 = _oracle(b)
    G = spec.num_q_heads // spec.num_kv_heads
    kc = b.k_cache.repeat_interleave(G, dim=1).contiguous()
    vc = b.v_cache.repeat_interleave(G, dim=1).contiguous()
    P, D, Hq = spec.page_size, spec.head_dim, spec.num_q_heads
    out1, lse1 = oracle.verify_attention(b.q, kc, vc, (Hq * P * D, P * D, D), b.block_table, b.seq_lens,
                                         b.q_indptr, Hq, P, b.num_pages)
    assert torch.equal(out0, out1) and torch.equal(lse0, lse1)


def test_poison_is_never_read_and_errors_are_reported():
    b = W.generate(W.scaled(W.CONFIGS[4], batch=5, ctx_div=64, vocab=32))
    out, _ = _oracle(b)
    assert out.abs().max() < 50.0          # poison is 1e4: any read of it would show
    bad = b.clone()
    bad.seq_lens[0] = bad.k_host[0]        # L < k+1
    with pytest.raises(oracle.OracleError) as e:
        _oracle(bad)
    assert e.value.code == oracle.ERR_LEN
    bad = b.clone()
    bad.block_table[1, 0] = b.num_pages
    with pytest.raises(oracle.OracleError) as e:
        _oracle(bad)
    assert e.value.code == oracle.ERR_PAGE


def test_req_list_subset_matches_full():
    b = W.generate(W.CONFIGS[0])
    full, lse = _oracle(b)
    part, lse_p = _oracle(b, req_list=[2])
    q0, m = int(b.q_indptr[2]), b.k_host[2] + 1
    assert torch.equal(part[q0:q0 + m], full[q0:q0 + m])
    assert torch.isnan(part[:q0]).all()


@pytest.mark.parametrize("ctx,page", [(4096, 16), (32768, 32)])
def test_the_parity_gates_catch_a_lost_page(ctx, page):
    """The tolerances of the GPU parity tests, tried on the oracle alone: a result computed without
    one middle page of the cache must fail them although it stays inside the contract's 2e-2 bound on
    the output (closed form: leaving P of L tokens out of a softmax over N(0,1) scores lowers LSE by
    about P/L, and the bf16 LSE gate is 2e-5)."""
    import dataclasses
    import parity_util
    spec = dataclasses.replace(W.CONFIGS[3], batch=1, num_q_heads=4, num_kv_heads=1, page_size=page, vocab=64,
                               ctx=("const", ctx), k=("const", 3), name="lost-page-cpu")
    b = W.generate(spec)
    ref_o, ref_l = _oracle(b)
    lost = b.clone()
    npages = ctx // page
    drop = npages // 2
    lost.block_table[0, drop:npages - 1] = b.block_table[0, drop + 1:npages]
    lost.seq_lens[0] -= page
    out, lse = _oracle(lost)
    shift = float((ref_l - lse).mean())
    assert 0.3 * page / ctx < shift < 3.0 * page / ctx
    assert float((out - ref_o).abs().max()) < 2e-2
    parity_util.check_attention(b, ref_o, ref_l, ref_o, ref_l)
    with pytest.raises(AssertionError):
        parity_util.check_attention(b, out, lse, ref_o, ref_l)
