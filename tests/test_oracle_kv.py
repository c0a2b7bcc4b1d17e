"""Pins for the oracle's cache-maintenance functions (CPU only): torch's indexed scatter on the
pool, bit-identity of untouched slots, composition with the pinned attention oracle, closed form
of the rolled-back lengths."""
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
