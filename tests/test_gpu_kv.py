"""GPU parity of the cache-maintenance calls: bit-exact against the oracle (pure copies and
integer arithmetic), at small and at benchmark sizes, plus append -> attend -> sample -> rollback
as one sequence."""
import dataclasses

import pytest
import torch

import oracle
import spx_workloads as W
import paper_2609_34370_b200 as spx

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _new_kv(b, seed, device="cpu"):
    g = torch.Generator().manual_seed(seed)
    s = b.spec
    shape = (b.total_q, s.num_kv_heads, s.head_dim)
    return (torch.randn(shape, generator=g).to(b.q.dtype).to(device), torch.randn(shape, generator=g).to(b.q.dtype).to(device))


@pytest.mark.parametrize("layout", ["HND", "NHD"])
@pytest.mark.parametrize("idx", [0, 1, 3, 4])
def test_append_is_bit_exact(idx, layout):
    spec = W.CONFIGS[idx] if idx == 0 else W.scaled(W.CONFIGS[idx], batch=9, ctx_div=16, vocab=64)
    b_cpu = W.generate(spec, layout=layout)
    nk, nv = _new_kv(b_cpu, 5)
    b = b_cpu.to(DEV)
    status = spx.kv_append(nk.to(DEV), nv.to(DEV), b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens,
                           b.q_indptr, spec.page_size, b.num_pages)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    oracle.kv_append(nk, nv, b_cpu.k_cache, b_cpu.v_cache, b_cpu.kv_strides, b_cpu.block_table, b_cpu.seq_lens,
                     b_cpu.q_indptr, spec.page_size, b_cpu.num_pages)
    assert torch.equal(b.k_cache.cpu(), b_cpu.k_cache) and torch.equal(b.v_cache.cpu(), b_cpu.v_cache)


def test_append_full_size_and_faults():
    spec = W.CONFIGS[1]
    b = W.generate(spec, device=DEV)
    nk, nv = _new_kv(b, 9, DEV)
    k_before = b.k_cache.clone()
    status = spx.kv_append(nk, nv, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                           spec.page_size, b.num_pages)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    b_cpu = dataclasses.replace(b.to("cpu"), k_cache=k_before.cpu())
    v_ref = b_cpu.v_cache.clone()          # V was appended on the device already: rebuild the reference from K only
    oracle.kv_append(nk.cpu(), nv.cpu(), b_cpu.k_cache, v_ref, b_cpu.kv_strides, b_cpu.block_table, b_cpu.seq_lens,
                     b_cpu.q_indptr, spec.page_size, b_cpu.num_pages)
    assert torch.equal(b.k_cache.cpu(), b_cpu.k_cache)
    assert torch.equal(b.v_cache.cpu(), v_ref)
    # a bad page id and a bad length are reported, the other requests are still written
    bad = W.generate(W.scaled(spec, batch=4, ctx_div=16, vocab=64)).to(DEV)
    nk, nv = _new_kv(bad, 2, DEV)
    last = (bad.seq_lens_host[1] - 1) // spec.page_size
    bad.block_table[1, last] = bad.num_pages + 3
    bad.seq_lens[2] = 1
    k0 = bad.k_cache.clone()
    status = spx.kv_append(nk, nv, bad.k_cache, bad.v_cache, bad.kv_strides, bad.block_table, bad.seq_lens,
                           bad.q_indptr, spec.page_size, bad.num_pages)
    torch.cuda.synchronize()
    assert int(status.item()) == (spx.DEV_BAD_PAGE | spx.DEV_BAD_LEN)
    assert not torch.equal(bad.k_cache, k0)


def test_rollback_and_whole_sequence():
    spec = W.scaled(W.CONFIGS[4], batch=16, ctx_div=16, vocab=4000)
    b_cpu = W.generate(spec)
    b = b_cpu.to(DEV)
    nk, nv = _new_kv(b_cpu, 7)
    spx.kv_append(nk.to(DEV), nv.to(DEV), b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                  spec.page_size, b.num_pages)
    out, lse, _ = spx.verify_attention(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                                       spec.num_kv_heads, spec.page_size, b.num_pages)
    acc, tok, _, _ = spx.rejection_sample(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample)
    new_len, status = spx.kv_rollback(b.seq_lens, b.q_indptr, acc)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # oracle: same sequence
    oracle.kv_append(nk, nv, b_cpu.k_cache, b_cpu.v_cache, b_cpu.kv_strides, b_cpu.block_table, b_cpu.seq_lens,
                     b_cpu.q_indptr, spec.page_size, b_cpu.num_pages)
    ref_o, _ = oracle.verify_attention(b_cpu.q, b_cpu.k_cache, b_cpu.v_cache, b_cpu.kv_strides, b_cpu.block_table,
                                       b_cpu.seq_lens, b_cpu.q_indptr, spec.num_kv_heads, spec.page_size, b_cpu.num_pages)
    ref = oracle.rejection_sample(b_cpu.target_logits, b_cpu.draft_logits, b_cpu.draft_ids, b_cpu.q_indptr,
                                  b_cpu.u_accept, b_cpu.u_sample)
    assert float((out.cpu().double() - ref_o).abs().max()) <= 2e-2
    assert torch.equal(acc.cpu(), ref.accepted_len)
    assert torch.equal(new_len.cpu(), oracle.kv_rollback(b_cpu.seq_lens, b_cpu.q_indptr, ref.accepted_len))
    # invalid accepted lengths are flagged
    bad_acc = acc.clone()
    bad_acc[0] = 99
    new_len, status = spx.kv_rollback(b.seq_lens, b.q_indptr, bad_acc)
    torch.cuda.synchronize()
    assert int(status.item()) == spx.DEV_BAD_LEN and int(new_len[0]) == -1


@pytest.mark.parametrize("layout", ["HND", "NHD"])
@pytest.mark.parametrize("idx,base", [(0, 10000.0), (1, 500000.0), (3, 1000000.0), (4, 500000.0)])
def test_append_with_rope_matches_oracle(idx, base, layout):
    """K rows rotated to their absolute positions on the way into the cache, Q rows in place, V
    copied.  Both sides compute in float64 and round float64 -> binary32 -> element type, so the
    stored values agree bit for bit up to the last bit of the two libraries' sin / cos / pow: at
    most one element in 10^4 may differ, and then by one unit in the last place."""
    spec = W.CONFIGS[idx] if idx == 0 else W.scaled(W.CONFIGS[idx], batch=9, ctx_div=4 if idx == 3 else 16, vocab=64)
    b_cpu = W.generate(spec, layout=layout)
    nk, nv = _new_kv(b_cpu, 5)
    b = b_cpu.to(DEV)
    q_dev = b.q.clone()
    status = spx.kv_append(nk.to(DEV), nv.to(DEV), b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens,
                           b.q_indptr, spec.page_size, b.num_pages, rope_base=base, q_rows=q_dev)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    oracle.kv_append(nk, nv, b_cpu.k_cache, b_cpu.v_cache, b_cpu.kv_strides, b_cpu.block_table, b_cpu.seq_lens,
                     b_cpu.q_indptr, spec.page_size, b_cpu.num_pages, rope_base=base)
    assert torch.equal(b.v_cache.cpu(), b_cpu.v_cache)
    pos = oracle.new_positions(b_cpu.seq_lens, b_cpu.q_indptr)
    q_ref = oracle.round_to(oracle.rope(b_cpu.q, pos, base), b_cpu.q.dtype)

    def close_to_the_last_bit(got, ref):
        got, ref = got.cpu(), ref
        if torch.equal(got, ref):
            return
        bits = torch.int16 if got.dtype == torch.bfloat16 else torch.int32
        d = (got.view(bits).to(torch.int64) - ref.view(bits).to(torch.int64)).abs()
        assert int(d.max()) <= 1 and float((d > 0).double().mean()) <= 1e-4, (int(d.max()), float((d > 0).double().mean()))

    close_to_the_last_bit(b.k_cache, b_cpu.k_cache)
    close_to_the_last_bit(q_dev, q_ref)
    assert not torch.equal(q_dev.cpu(), b_cpu.q)               # the rows were rotated
    # rope off: q_rows is left alone and the copy is the plain one
    q2 = b.q.clone()
    spx.kv_append(nk.to(DEV), nv.to(DEV), b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                  spec.page_size, b.num_pages, rope_base=0.0, q_rows=q2)
    torch.cuda.synchronize()
    assert torch.equal(q2, b.q)


def test_rope_arguments_are_validated():
    spec = W.CONFIGS[0]
    b = W.generate(spec).to(DEV)
    nk, nv = _new_kv(b, 1, DEV)
    for bad in (-1.0, float("nan"), float("inf")):
        with pytest.raises(spx.SpxError):
            spx.kv_append(nk, nv, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                          spec.page_size, b.num_pages, rope_base=bad)
