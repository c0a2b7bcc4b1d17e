"""Sanity of the seeded input generators (CPU only): shapes, page tables, poison, determinism."""
import torch

import spx_workloads as W


def test_generator_is_deterministic_and_well_formed():
    spec = W.scaled(W.CONFIGS[4], batch=9, ctx_div=32, vocab=128)
    a, b = W.generate(spec), W.generate(spec)
    for name in W.VerifyBatch._TENSORS:
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    P = spec.page_size
    used = set()
    for r, L in enumerate(a.seq_lens_host):
        n = (L + P - 1) // P
        row = a.block_table[r]
        assert (row[:n] >= 0).all() and (row[:n] < a.num_pages).all() and (row[n:] == -1).all()
        used.update(row[:n].tolist())
        assert L >= a.k_host[r] + 1
        if L % P:
            last = int(row[n - 1])
            assert (a.k_cache[last, :, L % P:, :] == W.POISON).all()
            assert (a.v_cache[last, :, L % P:, :] == -W.POISON).all()
    assert len(used) == sum((L + P - 1) // P for L in a.seq_lens_host)       # no page shared
    assert a.num_pages == 2 * len(used)                                       # fragmented pool
    unused = sorted(set(range(a.num_pages)) - used)
    assert (a.k_cache[unused] == W.POISON).all()
    assert set(a.k_host) <= {0, 2, 4, 6}
    assert a.q_indptr.tolist() == [0] + torch.tensor([k + 1 for k in a.k_host]).cumsum(0).tolist()
    assert a.draft_ids.numel() == a.total_d and ((a.draft_ids >= 0) & (a.draft_ids < spec.vocab)).all()
    assert ((a.u_accept >= 0) & (a.u_accept < 1)).all() and ((a.u_sample >= 0) & (a.u_sample < 1)).all()
    assert torch.equal(a.u_sample * 2 ** 24, torch.floor(a.u_sample * 2 ** 24))


def test_named_workloads_have_the_stated_shapes():
    c = W.CONFIGS
    assert [s.batch for s in c] == [4, 64, 128, 16, 256]
    assert [(s.num_q_heads, s.num_kv_heads, s.head_dim, s.page_size) for s in c] == \
        [(8, 2, 64, 16), (32, 8, 128, 16), (64, 8, 128, 16), (32, 8, 128, 32), (32, 8, 128, 16)]
    assert [s.vocab for s in c] == [1024, 128256, 128256, 32000, 128256]
    b = W.generate(c[0])
    assert b.q.dtype == torch.float32 and b.total_q == 20 and b.total_d == 16
    assert all(32 <= L <= 256 for L in b.seq_lens_host)


def test_nhd_layout_holds_the_same_values():
    spec = W.scaled(W.CONFIGS[0], batch=2)
    a, b = W.generate(spec, layout="HND"), W.generate(spec, layout="NHD")
    assert a.kv_strides != b.kv_strides and b.k_cache.shape[1] == spec.page_size
