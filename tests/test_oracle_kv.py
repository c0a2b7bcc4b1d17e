"""Pins for the oracle's cache-maintenance functions (CPU only): torch's indexed scatter on the
pool, bit-identity of untouched slots, composition with the pinned attention oracle, closed form
of the rolled-back lengths."""
import numpy as np
import pytest
import torch

import oracle
import spx_workloads as W


def _new_kv(b, seed):
    g = torch.Generator().manual_seed(seed)
    s = b.spec
    shape = (b.total_q, s.num_kv_heads, s.head_dim)
    return (torch.randn(shape, generator=g).to(b.q.dtype), torch.randn(shape, generator=g).to(b.q.dtype))


@pytest.mark.parametrize("layout", ["HND", "NHD"])
@pytest.mark.parametrize("cfg", [0, 4])
def test_append_matches_indexed_scatter_and_touches_nothing_else(cfg, layout):
    spec = W.CONFIGS[cfg] if cfg == 0 else W.scaled(W.CONFIGS[cfg], batch=7, ctx_div=32, vocab=64)
    b = W.generate(spec, layout=layout)
    nk, nv = _new_kv(b, 3)
    k0, v0 = b.k_cache.clone(), b.v_cache.clone()
    oracle.kv_append(nk, nv, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                     spec.page_size, b.num_pages)
    # library scatter on a copy: pool[page, :, slot, :] = new rows (HND) / pool[page, slot, :, :] (NHD)
    ek, ev = k0.clone(), v0.clone()
    P = spec.page_size
    qi = b.q_indptr.tolist()
    for r, L in enumerate(b.seq_lens_host):
        m = b.k_host[r] + 1
        t = torch.arange(L - m, L)
        pages = b.block_table[r, (t // P).long()].long()
        slots = (t % P).long()
        if layout == "HND":
            ek[pages, :, slots, :] = nk[qi[r]:qi[r] + m]
            ev[pages, :, slots, :] = nv[qi[r]:qi[r] + m]
        else:
            ek[pages, slots, :, :] = nk[qi[r]:qi[r] + m]
            ev[pages, slots, :, :] = nv[qi[r]:qi[r] + m]
    assert torch.equal(b.k_cache, ek) and torch.equal(b.v_cache, ev)
    changed = (b.k_cache != k0).any(dim=-1)
    assert int(changed.sum()) <= b.total_q * spec.num_kv_heads          # only the new (token, head) rows moved


def test_append_then_attend_equals_attending_a_prefilled_cache():
    b = W.generate(W.CONFIGS[0])
    s = b.spec
    ref_o, ref_l = oracle.verify_attention(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens,
                                           b.q_indptr, s.num_kv_heads, s.page_size, b.num_pages)
    # cut the new positions out of the cache, poison their slots, append them back
    P = s.page_size
    nk = torch.empty(b.total_q, s.num_kv_heads, s.head_dim)
    nv = torch.empty_like(nk)
    b2 = b.clone()
    qi = b.q_indptr.tolist()
    for r, L in enumerate(b.seq_lens_host):
        m = b.k_host[r] + 1
        for j in range(m):
            t = L - m + j
            page, slot = int(b.block_table[r, t // P]), t % P
            nk[qi[r] + j] = b.k_cache[page, :, slot, :]
            nv[qi[r] + j] = b.v_cache[page, :, slot, :]
            b2.k_cache[page, :, slot, :] = W.POISON
            b2.v_cache[page, :, slot, :] = -W.POISON
    oracle.kv_append(nk, nv, b2.k_cache, b2.v_cache, b2.kv_strides, b2.block_table, b2.seq_lens, b2.q_indptr, P,
                     b2.num_pages)
    o, l = oracle.verify_attention(b2.q, b2.k_cache, b2.v_cache, b2.kv_strides, b2.block_table, b2.seq_lens,
                                   b2.q_indptr, s.num_kv_heads, s.page_size, b2.num_pages)
    assert torch.equal(o, ref_o) and torch.equal(l, ref_l)


def test_append_errors():
    b = W.generate(W.CONFIGS[0])
    nk, nv = _new_kv(b, 1)
    bad = b.clone()
    bad.seq_lens[2] = 2
    with pytest.raises(oracle.OracleError) as e:
        oracle.kv_append(nk, nv, bad.k_cache, bad.v_cache, bad.kv_strides, bad.block_table, bad.seq_lens,
                         bad.q_indptr, b.spec.page_size, b.num_pages)
    assert e.value.code == oracle.ERR_LEN
    bad = b.clone()
    last = (b.seq_lens_host[1] - 1) // b.spec.page_size
    bad.block_table[1, last] = -1
    with pytest.raises(oracle.OracleError) as e:
        oracle.kv_append(nk, nv, bad.k_cache, bad.v_cache, bad.kv_strides, bad.block_table, bad.seq_lens,
                         bad.q_indptr, b.spec.page_size, b.num_pages)
    assert e.value.code == oracle.ERR_PAGE


def test_rollback_closed_form_and_round_trip():
    qi = torch.tensor([0, 5, 6, 10, 17], dtype=torch.int32)        # k = 4, 0, 3, 6
    L = torch.tensor([100, 7, 40, 9], dtype=torch.int32)
    for n in ([0, 0, 0, 0], [4, 0, 3, 6], [2, 0, 1, 5]):
        out = oracle.kv_rollback(L, qi, torch.tensor(n, dtype=torch.int32))
        k = (qi[1:] - qi[:-1] - 1)
        assert out.tolist() == (L - (k - torch.tensor(n, dtype=torch.int32))).tolist()
    assert oracle.kv_rollback(L, qi, torch.tensor([4, 0, 3, 6], dtype=torch.int32)).tolist() == L.tolist()
    assert oracle.kv_rollback(L, qi, torch.zeros(4, dtype=torch.int32)).tolist() == [96, 7, 37, 3]
    with pytest.raises(oracle.OracleError):
        oracle.kv_rollback(L, qi, torch.tensor([5, 0, 0, 0], dtype=torch.int32))
    with pytest.raises(oracle.OracleError):
        oracle.kv_rollback(L, qi, torch.tensor([0, 0, -1, 0], dtype=torch.int32))


# ---- rotary embedding (the optional fusion of the append) ----------------------------------------
# Pinned to what the rotation is by definition: a hand-worked pair, the identity at position 0,
# a complex-multiplication restatement, length preservation, additivity of positions and the
# relative-position property of rotated dot products.

def test_rope_hand_worked_pair_and_identity():
    # D = 2: one pair, frequency base^0 = 1, angle = position.  (1, 0) at position 1 -> (cos 1, sin 1).
    x = torch.tensor([[[1.0, 0.0]], [[0.0, 2.0]], [[3.0, 4.0]]], dtype=torch.float32)
    y = oracle.rope(x, torch.tensor([1, 1, 0], dtype=torch.int32), 10000.0)
    assert y[0, 0].tolist() == pytest.approx([0.5403023058681398, 0.8414709848078965], abs=1e-15)
    assert y[1, 0].tolist() == pytest.approx([-2 * 0.8414709848078965, 2 * 0.5403023058681398], abs=1e-15)
    assert y[2, 0].tolist() == [3.0, 4.0]                      # position 0: untouched
    # D = 4, base 100: pair 0 turns by t, pair 1 by t / 10 (base^(-2/4) = 0.1)
    x = torch.tensor([[[1.0, 1.0, 0.0, 0.0]]], dtype=torch.float32)
    y = oracle.rope(x, torch.tensor([5], dtype=torch.int32), 100.0)[0, 0]
    assert y.tolist() == pytest.approx([np.cos(5.0), np.cos(0.5), np.sin(5.0), np.sin(0.5)], abs=1e-15)


def test_rope_equals_complex_multiplication_and_preserves_length():
    g = torch.Generator().manual_seed(5)
    rows, H, D, base = 9, 3, 64, 500000.0
    x = torch.randn(rows, H, D, generator=g, dtype=torch.float32)
    pos = torch.tensor([0, 1, 2, 17, 255, 4096, 32767, 100000, 7], dtype=torch.int32)
    y = oracle.rope(x, pos, base).numpy()
    xd = x.double().numpy()
    z = xd[..., :D // 2] + 1j * xd[..., D // 2:]
    inv_freq = base ** (-np.arange(D // 2) * 2.0 / D)
    w = np.exp(1j * pos.numpy()[:, None, None].astype(np.float64) * inv_freq[None, None, :])
    ref = z * w
    assert np.allclose(y[..., :D // 2], ref.real, rtol=0, atol=1e-9)
    assert np.allclose(y[..., D // 2:], ref.imag, rtol=0, atol=1e-9)
    assert np.allclose((y ** 2).sum(-1), (xd ** 2).sum(-1), rtol=1e-12)


def test_rope_positions_add_and_dot_products_depend_on_the_offset_only():
    g = torch.Generator().manual_seed(6)
    H, D, base = 2, 32, 10000.0
    q = torch.randn(1, H, D, generator=g, dtype=torch.float32)
    k = torch.randn(1, H, D, generator=g, dtype=torch.float32)
    def at(x, t):
        return oracle.rope(x, torch.tensor([t], dtype=torch.int32), base)
    # R(a) R(b) = R(a + b): rotate the float64 result again (fed back as float32 loses 1e-7)
    once = at(q, 300)
    twice = oracle.rope(at(q, 100).to(torch.float32), torch.tensor([200], dtype=torch.int32), base)
    assert torch.allclose(once, twice, atol=1e-5)
    # <R(m) q, R(n) k> is a function of m - n
    d1 = (at(q, 1000) * at(k, 990)).sum(-1)
    d2 = (at(q, 50) * at(k, 40)).sum(-1)
    d3 = (at(q, 10) * k.double()).sum(-1)
    assert torch.allclose(d1, d2, atol=1e-9) and torch.allclose(d1, d3, atol=1e-9)


def test_kv_append_with_rope_rotates_k_only():
    spec = W.scaled(W.CONFIGS[1], batch=3, ctx_div=16, vocab=64)
    b = W.generate(spec)
    g = torch.Generator().manual_seed(8)
    nk = torch.randn(b.total_q, spec.num_kv_heads, spec.head_dim, generator=g).to(b.k_cache.dtype)
    nv = torch.randn(b.total_q, spec.num_kv_heads, spec.head_dim, generator=g).to(b.k_cache.dtype)
    k1, v1 = b.k_cache.clone(), b.v_cache.clone()
    k2, v2 = b.k_cache.clone(), b.v_cache.clone()
    oracle.kv_append(nk, nv, k1, v1, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr, spec.page_size, b.num_pages)
    oracle.kv_append(nk, nv, k2, v2, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr, spec.page_size, b.num_pages,
                     rope_base=500000.0)
    assert torch.equal(v1, v2)                                   # V is copied as it is
    pos = oracle.new_positions(b.seq_lens, b.q_indptr)
    rot = oracle.round_to(oracle.rope(nk, pos, 500000.0), nk.dtype)
    k3 = b.k_cache.clone()
    oracle.kv_append(rot, nv, k3, v1.clone(), b.kv_strides, b.block_table, b.seq_lens, b.q_indptr, spec.page_size,
                     b.num_pages)
    assert torch.equal(k2, k3) and not torch.equal(k1, k2)
    # positions: the new rows of request r are its last k_r + 1 tokens
    qi, sl = b.q_indptr.tolist(), b.seq_lens.tolist()
    for r in range(b.batch):
        assert pos[qi[r]:qi[r + 1]].tolist() == list(range(sl[r] - (qi[r + 1] - qi[r]), sl[r]))
