"""The host-buffer entry point and the no-workspace entry point give the same bits as the device
path, with and without per-request sampling parameters (the device path itself is held against
the oracle elsewhere)."""
import pytest
import torch

import spx_workloads as W
import paper_2609_34370_b200 as spx

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _device_step(b, spec, **extra):
    out = torch.empty_like(b.q)
    lse = torch.empty(b.q.shape[:2], dtype=torch.float32, device=DEV)
    acc = torch.empty(b.batch, dtype=torch.int32, device=DEV)
    tok = torch.empty(b.total_q, dtype=torch.int32, device=DEV)
    a = spx.make_attn_args(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                           spec.num_kv_heads, spec.page_size, b.num_pages, out, lse, 0.0, max(b.k_host) + 1)
    s = spx.make_sample_args(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample, acc, tok,
                             None, None, extra.get("temperature"), extra.get("top_k"), extra.get("top_p"))
    ws = spx.Workspace.allocate(spx.workspace_size(a, s), DEV)
    spx.verify_step(a, s, ws, DEV)
    torch.cuda.synchronize()
    return out, lse, acc, tok, int(ws.status.item())


@pytest.mark.parametrize("variant", ["base", "temperature", "filters"])
@pytest.mark.parametrize("idx", [0, 1, 4])
def test_host_step_equals_device_step(idx, variant):
    spec = W.CONFIGS[idx] if idx == 0 else W.scaled(W.CONFIGS[idx], batch=12, ctx_div=16, vocab=9000)
    b_cpu = W.generate(spec)
    B = b_cpu.batch
    extra_cpu = {}
    if variant != "base":
        extra_cpu["temperature"] = torch.tensor([[1.0, 0.0, 0.6, 1.8][r % 4] for r in range(B)])
    if variant == "filters":
        extra_cpu["top_k"] = torch.tensor([[0, 40, 1, 0][r % 4] for r in range(B)], dtype=torch.int32)
        extra_cpu["top_p"] = torch.tensor([[0.9, 1.0, 1.0, 0.5][r % 4] for r in range(B)])
    b = b_cpu.to(DEV)
    out, lse, acc, tok, status = _device_step(b, spec, **{k: v.to(DEV) for k, v in extra_cpu.items()})
    assert status & ~spx.DEV_DEGENERATE == 0
    # host path: every tensor pinned on the host
    pin = {n: getattr(b_cpu, n).pin_memory() for n in W.VerifyBatch._TENSORS}
    extra_pin = {k: v.pin_memory() for k, v in extra_cpu.items()}
    out_h = torch.empty(out.shape, dtype=out.dtype).pin_memory()
    lse_h = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
    acc_h = torch.empty(B, dtype=torch.int32).pin_memory()
    tok_h = torch.empty(b_cpu.total_q, dtype=torch.int32).pin_memory()
    st_h = torch.zeros(1, dtype=torch.int32).pin_memory()
    ah = spx.make_attn_args(pin["q"], pin["k_cache"], pin["v_cache"], b_cpu.kv_strides, pin["block_table"], pin["seq_lens"],
                            pin["q_indptr"], spec.num_kv_heads, spec.page_size, b_cpu.num_pages, out_h, lse_h, 0.0, max(b_cpu.k_host) + 1)
    sh = spx.make_sample_args(pin["target_logits"], pin["draft_logits"], pin["draft_ids"], pin["q_indptr"], pin["u_accept"],
                              pin["u_sample"], acc_h, tok_h, None, None, extra_pin.get("temperature"), extra_pin.get("top_k"),
                              extra_pin.get("top_p"))
    pool_elems = b_cpu.k_cache.numel()
    arena = torch.empty(spx.host_step_arena_size(ah, sh, pool_elems), dtype=torch.uint8, device=DEV)
    spx.verify_step_host(ah, sh, pool_elems, arena, st_h, DEV)
    torch.cuda.synchronize()
    assert int(st_h.item()) & ~spx.DEV_DEGENERATE == 0
    assert torch.equal(out_h, out.cpu()) and torch.equal(lse_h, lse.cpu())
    assert torch.equal(acc_h, acc.cpu()) and torch.equal(tok_h, tok.cpu())


def test_static_scratch_entry_point_takes_the_variants():
    spec = W.scaled(W.CONFIGS[1], batch=10, ctx_div=16, vocab=12000)
    b = W.generate(spec, device=DEV)
    B = b.batch
    tau = torch.tensor([[1.0, 0.0, 0.6, 1.8][r % 4] for r in range(B)], device=DEV)
    tk = torch.tensor([[0, 40, 1, 0][r % 4] for r in range(B)], dtype=torch.int32, device=DEV)
    tp = torch.tensor([[0.9, 1.0, 1.0, 0.5][r % 4] for r in range(B)], device=DEV)
    acc, tok, _, ws = spx.rejection_sample(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample,
                                           temperature=tau, top_k=tk, top_p=tp)
    acc2 = torch.empty_like(acc)
    tok2 = torch.empty_like(tok)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    s = spx.make_sample_args(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample, acc2, tok2,
                             None, None, tau, tk, tp)
    import ctypes as C
    lib = spx.load_library()
    code = lib.spx_rejection_sample_static(C.byref(s), status.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert code == 0 and int(status.item()) & ~spx.DEV_DEGENERATE == 0
    assert torch.equal(acc, acc2) and torch.equal(tok, tok2)
