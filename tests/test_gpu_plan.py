"""Invariants of the attention work plan, read back from the workspace after a call.

The plan cuts the 128-token tiles of all (request, kv head) pairs, in (request, head) order, into
one contiguous range per CTA.  Whatever the length mix, every tile of every valid pair must be
covered exactly once, a CTA's entries must be consecutive on the tile axis, a pair that several
entries cover must own distinct partial slots, and the ranges must carry about the same load.
"""
import dataclasses

import numpy as np
import pytest
import torch

import spx_workloads as W
import paper_2609_34370_b200 as spx
from paper_2609_34370_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TILE = 128


def _plan_of(b, break_requests=()):
    s = b.spec
    b = b.to(DEV)
    seq_lens = b.seq_lens.clone()
    for r in break_requests:                     # invalid request: context shorter than its query rows
        seq_lens[r] = 0
    out = torch.empty_like(b.q)
    lse = torch.empty(b.q.shape[:2], dtype=torch.float32, device=DEV)
    a = binding.make_attn_args(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, seq_lens, b.q_indptr,
                               s.num_kv_heads, s.page_size, b.num_pages, out, lse)
    lay = spx.plan_layout(a)
    ws = spx.Workspace.allocate(spx.workspace_size(a, None), DEV)
    assert lay["attn_bytes"] <= ws.buf.numel()
    spx.verify_attention(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, seq_lens, b.q_indptr,
                         s.num_kv_heads, s.page_size, b.num_pages, out=out, lse=lse, ws=ws)
    torch.cuda.synchronize()
    raw = ws.buf.cpu().numpy()
    hdr = raw[lay["header"]:lay["header"] + 32].view(np.int32)
    n_work, n_cta, n_slots, total_tiles, _, overflow = (int(v) for v in hdr[:6])
    cta_off = raw[lay["cta_off"]:lay["cta_off"] + 4 * (n_cta + 1)].view(np.int32)
    work = raw[lay["work"]:lay["work"] + 32 * n_work].view(np.int32).reshape(-1, 8)
    pairs = b.batch * s.num_kv_heads
    nch = raw[lay["pair_nchunks"]:lay["pair_nchunks"] + 4 * pairs].view(np.int32)
    base = raw[lay["pair_part_base"]:lay["pair_part_base"] + 4 * pairs].view(np.int32)
    return dict(n_work=n_work, n_cta=n_cta, n_slots=n_slots, total_tiles=total_tiles, overflow=overflow, cta_off=cta_off,
                work=work, nch=nch, base=base, lay=lay, seq_lens=seq_lens.cpu().numpy(), status=int(ws.status.item()))


def _check_plan(b, P, invalid=()):
    Hkv = b.spec.num_kv_heads
    tiles = [0 if r in invalid else (int(L) + TILE - 1) // TILE for r, L in enumerate(P["seq_lens"])]
    assert P["overflow"] == 0
    assert P["total_tiles"] == sum(tiles)
    assert P["n_work"] <= P["lay"]["max_work"] and P["n_slots"] <= P["lay"]["max_part_slots"]
    assert P["cta_off"][0] == 0 and P["cta_off"][P["n_cta"]] == P["n_work"]
    assert (np.diff(P["cta_off"]) >= 0).all()
    prefix = np.concatenate([[0], np.cumsum(tiles)])
    covered = {}
    slots = set()
    loads = []
    axis_pos = -1
    for c in range(P["n_cta"]):
        ents = P["work"][P["cta_off"][c]:P["cta_off"][c + 1]]
        load = 0
        for req, tb, te, slot, q0, m, L, g in ents:
            assert 0 <= req < b.batch and 0 <= g < Hkv and req not in invalid
            assert 0 <= tb < te <= tiles[req]
            assert q0 == int(b.q_indptr[req]) and m == int(b.q_indptr[req + 1]) - q0 and L == int(P["seq_lens"][req])
            # entries follow the tile axis: (request, head, tile) strictly increasing over the whole list
            start = int(prefix[req]) * Hkv + g * tiles[req] + tb
            assert start > axis_pos
            axis_pos = start + (te - tb) - 1
            covered.setdefault((req, g), []).append((tb, te, slot))
            if slot >= 0:
                assert slot < P["n_slots"] and slot not in slots
                slots.add(slot)
            load += te - tb
        loads.append(load)
    for r in range(b.batch):
        for g in range(Hkv):
            pair = r * Hkv + g
            chunks = sorted(covered.get((r, g), []))
            assert P["nch"][pair] == len(chunks)
            if tiles[r] == 0:
                assert not chunks
                continue
            assert chunks[0][0] == 0 and chunks[-1][1] == tiles[r]
            assert all(chunks[i][1] == chunks[i + 1][0] for i in range(len(chunks) - 1))   # no gap, no overlap
            if len(chunks) == 1:
                assert chunks[0][2] == -1 and P["base"][pair] == -1
            else:
                assert [c[2] for c in chunks] == list(range(P["base"][pair], P["base"][pair] + len(chunks)))
    return loads


def test_plan_covers_every_tile_once_on_the_named_workloads():
    for idx in (1, 2, 4):
        b = W.generate(W.CONFIGS[idx])
        P = _plan_of(b)
        assert P["status"] == 0
        loads = _check_plan(b, P)
        split_pairs = int((P["nch"] > 1).sum())
        assert split_pairs <= P["n_cta"] - 1
        # equal cost, not equal tiles: a range of short pairs holds fewer tiles; still every range is
        # within a third of the mean and none is empty when there is enough work
        mean = sum(loads) / len(loads)
        assert min(loads) > 0.6 * mean and max(loads) < 1.34 * mean, (idx, min(loads), mean, max(loads))


@pytest.mark.parametrize("seed", range(6))
def test_plan_invariants_on_random_batches(seed):
    rng = np.random.default_rng(seed)
    batch = int(rng.choice([1, 2, 7, 40, 300, 1500]))
    hi = int(rng.choice([40, 700, 5000])) if batch >= 300 else int(rng.choice([40, 700, 5000, 30000]))
    hq, hkv = [(8, 2), (8, 4), (16, 2)][seed % 3]
    spec = dataclasses.replace(W.CONFIGS[1], batch=batch, num_q_heads=hq, num_kv_heads=hkv, head_dim=64, vocab=64,
                               ctx=("uniform", 8, hi), k=("choice", (0, 1, 3, 5)), name=f"plan-{seed}")
    b = W.generate(spec, seed=100 + seed)
    invalid = tuple(int(r) for r in rng.choice(batch, size=min(batch, 3), replace=False)) if seed % 2 else ()
    P = _plan_of(b, break_requests=invalid)
    assert (P["status"] != 0) == bool(invalid)          # invalid requests are reported, the rest is planned
    _check_plan(b, P, invalid=set(invalid))
