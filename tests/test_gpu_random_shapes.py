"""Seeded sweep over shapes the named workloads do not visit: head counts, head sizes, page sizes,
ragged draft counts, both pool layouts, fragmented pools, both dtypes.  Each case is held against
the oracle with the tolerances of parity_util (attention) and bit-exactness outside the counted
near-tie classes (sampling); the whole step must agree with its two halves."""
import random

import pytest
import torch

import spx_workloads as W
import paper_2609_34370_b200 as spx
from parity_util import check_attention, check_sampling, gpu_attention, gpu_sample, oracle_attention

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
HEADS = [(8, 2), (16, 4), (32, 8), (8, 8), (64, 8), (4, 1), (12, 4)]


def _spec(seed: int) -> W.WorkloadSpec:
    rng = random.Random(seed)
    hq, hkv = rng.choice(HEADS)
    dtype = "fp32" if seed % 6 == 5 else "bf16"
    ks = tuple(sorted(set(rng.choice([0, 1, 2, 3, 4, 5, 7]) for _ in range(3))))
    hi = rng.choice([40, 300, 1500])
    return W.WorkloadSpec(
        name=f"random-{seed}", index=100 + seed, batch=rng.randint(1, 12), num_q_heads=hq, num_kv_heads=hkv,
        head_dim=rng.choice([64, 128]), page_size=rng.choice([8, 16, 32, 64]), vocab=rng.choice([1024, 5000, 32000]),
        dtype=dtype, ctx=("uniform", max(ks) + 1, max(ks) + 1 + hi), k=("choice", ks),
        sigma_d=rng.choice([0.5, 1.0, 2.0]), pool_factor=rng.choice([1, 2]))


@pytest.mark.parametrize("seed", range(24))
def test_random_shape(seed):
    spec = _spec(seed)
    layout = "NHD" if seed % 3 == 1 else "HND"
    b_cpu = W.generate(spec, layout=layout)
    b = b_cpu.to(DEV)
    out, lse, ws = gpu_attention(b, max_q_len=max(b.k_host) + 1)
    assert int(ws.status.item()) == 0, spec
    ref_o, ref_l = oracle_attention(b_cpu)
    check_attention(b_cpu, out, lse, ref_o, ref_l)
    acc, tok, _, ws2 = gpu_sample(b)
    assert int(ws2.status.item()) == 0
    rep = check_sampling(b_cpu, acc, tok)
    assert not rep.hard_mismatch, (spec, rep)
    # the composed step gives the same bits as its halves
    out2 = torch.empty_like(out)
    lse2 = torch.empty_like(lse)
    acc2, tok2 = torch.empty_like(acc), torch.empty_like(tok)
    a = spx.make_attn_args(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                           spec.num_kv_heads, spec.page_size, b.num_pages, out2, lse2, 0.0, max(b.k_host) + 1)
    s = spx.make_sample_args(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample, acc2, tok2)
    ws3 = spx.Workspace.allocate(spx.workspace_size(a, s), DEV)
    spx.verify_step(a, s, ws3, DEV)
    torch.cuda.synchronize()
    assert int(ws3.status.item()) == 0
    assert torch.equal(out, out2) and torch.equal(lse, lse2) and torch.equal(acc, acc2) and torch.equal(tok, tok2)


@pytest.mark.parametrize("seed", range(12))
def test_random_shape_with_random_sampling_parameters(seed):
    import dataclasses
    import oracle
    spec = dataclasses.replace(_spec(seed + 50), dtype="bf16")
    b_cpu = W.generate(spec)
    rng = random.Random(1000 + seed)
    B, V = b_cpu.batch, spec.vocab
    tau = torch.tensor([rng.choice([0.0, 0.5, 1.0, 1.7]) for _ in range(B)])
    tk = torch.tensor([rng.choice([0, 1, 10, 100]) for _ in range(B)], dtype=torch.int32)
    tp = torch.tensor([rng.choice([1.0, 0.9, 0.5]) for _ in range(B)])
    # harness side: most drafts are redrawn from the filtered draft law so that acceptances occur
    g = torch.Generator().manual_seed(seed)
    ids = b_cpu.draft_ids.clone()
    qi = b_cpu.q_indptr.tolist()
    for r in range(B):
        d0, k = qi[r] - r, qi[r + 1] - qi[r] - 1
        for i in range(k):
            if float(tau[r]) == 0.0:
                if rng.random() < 0.7:
                    ids[d0 + i] = int(torch.argmax(b_cpu.target_logits[qi[r] + i, :V].float()))
            elif rng.random() < 0.85:
                q, _, _ = oracle.filtered_row(b_cpu.draft_logits[d0 + i, :V], float(tau[r]), int(tk[r]), float(tp[r]))
                ids[d0 + i] = int(torch.multinomial(q, 1, generator=g))
    b_cpu = dataclasses.replace(b_cpu, draft_ids=ids)
    b = b_cpu.to(DEV)
    acc, tok, _, ws = spx.rejection_sample(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample,
                                           temperature=tau.to(DEV), top_k=tk.to(DEV), top_p=tp.to(DEV))
    torch.cuda.synchronize()
    assert int(ws.status.item()) & ~spx.DEV_DEGENERATE == 0
    rep = check_sampling(b_cpu, acc, tok, temperature=tau, top_k=tk, top_p=tp)
    assert not rep.hard_mismatch, (spec, rep, tau.tolist(), tk.tolist(), tp.tolist())
    # KV append of random new tokens, bit for bit
    gk = torch.Generator().manual_seed(seed + 7)
    shape = (b_cpu.total_q, spec.num_kv_heads, spec.head_dim)
    nk, nv = torch.randn(shape, generator=gk).to(b_cpu.q.dtype), torch.randn(shape, generator=gk).to(b_cpu.q.dtype)
    st = spx.kv_append(nk.to(DEV), nv.to(DEV), b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                       spec.page_size, b.num_pages)
    torch.cuda.synchronize()
    oracle.kv_append(nk, nv, b_cpu.k_cache, b_cpu.v_cache, b_cpu.kv_strides, b_cpu.block_table, b_cpu.seq_lens, b_cpu.q_indptr,
                     spec.page_size, b_cpu.num_pages)
    assert int(st.item()) == 0 and torch.equal(b.k_cache.cpu(), b_cpu.k_cache) and torch.equal(b.v_cache.cpu(), b_cpu.v_cache)
