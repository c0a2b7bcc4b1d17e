#!/usr/bin/env python
"""Benchmark of the speculative-decoding verify step (one step = attention + rejection sampling
for one batch of synthetic requests).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload I] [--impl reference]

Prints ONE JSON line.  `value` is verified tokens per second (sum over requests of accepted+1,
per step, over all GPUs) with inputs resident in HBM; `e2e` is the same metric through the
host-buffer entry point with host<->device copies inside the timed region; `roofline` is the
verify-attention kernel (the kernel that streams the KV cache) against the measured HBM copy
bandwidth; `cpu_baseline` is the float64 CPU oracle timed on a bounded sample of the same
workload.  With N > 1 (under torchrun) every rank runs an independent replica of the workload on
its own GPU (the path has no exchange step), times are the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import spx_workloads as W  # noqa: E402

METRIC = "verified_tokens_per_s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one verify-attention launch, from the ncu captures
# summarised in profiles/attention_traffic.txt (two launches each, averaged).  The mixed-length
# workload was captured on its first 64 requests (1186.8 MB for 1176.1 MB of KV) and scaled to the
# full batch by the KV bytes: the traffic beyond the KV bytes (query and output rows, block
# tables, partials of split pairs) grows with the batch like the KV bytes do.
NCU_TRAFFIC_BYTES = {"tiny-fp32": 0.621e6, "llama3-8b": 626.7e6, "llama3-70b": 761.1e6, "long-context": 2154.5e6,
                     "selective-mix": 4309.4e6}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if visible:
                entry = visible.split(",")[index]
                phys = int(entry) if entry.isdigit() else None
            self.h = (pynvml.nvmlDeviceGetHandleByIndex(phys) if phys is not None
                      else pynvml.nvmlDeviceGetHandleByUUID(entry))
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _poll(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while True:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            if self._stop.wait(0.002):
                break

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._poll, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


def reduce_over_ranks(ms: float, tokens: float, device) -> tuple:
    """Whole-job figures from per-rank ones: the slowest rank's time, the sum of the tokens.

    Each rank runs an independent replica, so this is the only communication of the benchmark.
    """
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    n = torch.tensor([tokens], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), float(n.item())


def sub_batch(b_cpu: W.VerifyBatch, n_req: int) -> W.VerifyBatch:
    """The first n_req requests of a host batch (KV pools shared, not copied)."""
    import dataclasses
    qi = b_cpu.q_indptr.tolist()
    tq, td = qi[n_req], qi[n_req] - n_req
    return dataclasses.replace(
        b_cpu, q=b_cpu.q[:tq], block_table=b_cpu.block_table[:n_req], seq_lens=b_cpu.seq_lens[:n_req],
        q_indptr=b_cpu.q_indptr[:n_req + 1], target_logits=b_cpu.target_logits[:tq],
        draft_logits=b_cpu.draft_logits[:td], draft_ids=b_cpu.draft_ids[:td], u_accept=b_cpu.u_accept[:td],
        u_sample=b_cpu.u_sample[:n_req], seq_lens_host=b_cpu.seq_lens_host[:n_req], k_host=b_cpu.k_host[:n_req])


def oracle_sample_size(spec: W.WorkloadSpec) -> int:
    """Requests in the CPU-baseline sample: about 10-30 s of float64 work on ~8-32 cores."""
    return {0: 4, 1: 64, 2: 128, 3: 4, 4: 64}.get(spec.index, min(spec.batch, 8))


def time_oracle(b_cpu: W.VerifyBatch, n_req: int):
    """One oracle pass over the sample.  Returns (seconds, verified tokens, threads)."""
    import oracle
    sb = sub_batch(b_cpu, n_req)
    s = sb.spec
    t0 = time.perf_counter()
    oracle.verify_attention(sb.q, sb.k_cache, sb.v_cache, sb.kv_strides, sb.block_table, sb.seq_lens, sb.q_indptr,
                            s.num_kv_heads, s.page_size, sb.num_pages)
    res = oracle.rejection_sample(sb.target_logits, sb.draft_logits, sb.draft_ids, sb.q_indptr, sb.u_accept,
                                  sb.u_sample)
    dt = time.perf_counter() - t0
    return dt, int(res.accepted_len.sum()) + n_req, oracle.num_threads()


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = W.CONFIGS[args.workload]
    b_cpu = W.generate(spec, device="cpu")
    n_req = oracle_sample_size(spec)
    for _ in range(args.warmup):
        time_oracle(b_cpu, n_req)
    total_t, tokens, threads = 0.0, 0, 1
    for _ in range(args.steps):
        dt, tok, threads = time_oracle(b_cpu, n_req)
        total_t += dt
        tokens += tok
    value = tokens / total_t
    sample = f"first {n_req} of {spec.batch} requests per step (attention + sampling, float64)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": spec.name, "batch": spec.batch, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def time_extras(spx, binding, spec, b, attn_args, dev, iters: int = 200):
    """Device time (CUDA events, mean of `iters` calls after 5 warm-up calls, L2 not flushed for the
    small ones: they are launch-bound) of the calls around the step and of the verification variants."""
    def timed(fn):
        nonlocal iters
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters * 1e3      # microseconds

    g = torch.Generator().manual_seed(spec.seed + 7)
    shape = (b.total_q, spec.num_kv_heads, spec.head_dim)
    new_k = torch.randn(shape, generator=g).to(b.q.dtype).to(dev)
    new_v = torch.randn(shape, generator=g).to(b.q.dtype).to(dev)
    k_pool, v_pool = b.k_cache.clone(), b.v_cache.clone()     # the benchmark's own pools stay untouched
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    acc = torch.empty(b.batch, dtype=torch.int32, device=dev)
    tok = torch.empty(b.total_q, dtype=torch.int32, device=dev)
    new_len = torch.empty_like(b.seq_lens)
    out = {}
    out["kv_append_us"] = timed(lambda: spx.kv_append(new_k, new_v, k_pool, v_pool, b.kv_strides, b.block_table, b.seq_lens,
                                                      b.q_indptr, spec.page_size, b.num_pages, status=status))
    out["kv_append_bytes"] = 2 * new_k.numel() * new_k.element_size() * 2
    q_rot = b.q.clone()
    out["kv_append_rope_us"] = timed(lambda: spx.kv_append(new_k, new_v, k_pool, v_pool, b.kv_strides, b.block_table, b.seq_lens,
                                                           b.q_indptr, spec.page_size, b.num_pages, status=status,
                                                           rope_base=500000.0, q_rows=q_rot))
    base = binding.make_sample_args(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample, acc, tok)
    ws = spx.Workspace.allocate(spx.workspace_size(attn_args, base), dev)
    lib = spx.load_library()
    import ctypes as C
    stream = torch.cuda.current_stream(dev).cuda_stream

    def sample_call(sargs):
        return lambda: lib.spx_rejection_sample(C.byref(sargs), ws.buf.data_ptr(), ws.buf.numel(), ws.status.data_ptr(), stream)

    out["sample_tau1_us"] = timed(sample_call(base))
    out["kv_rollback_us"] = timed(lambda: spx.kv_rollback(b.seq_lens, b.q_indptr, acc, out=new_len, status=status))
    taus = {"mixed": torch.tensor([[1.0, 0.0, 0.3, 0.7, 0.0, 1.5, 4.0, 0.05][r % 8] for r in range(b.batch)]),
            "0.7": torch.full((b.batch,), 0.7), "greedy": torch.zeros(b.batch)}
    for name, tau in taus.items():
        tau_d = tau.to(dev)
        sv = binding.make_sample_args(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample,
                                      acc, tok, None, None, tau_d)
        ws.ensure(spx.workspace_size(attn_args, sv))
        out[f"sample_tau_{name}_us"] = timed(sample_call(sv))
        out[f"step_tau_{name}_us"] = timed(lambda: spx.verify_step(attn_args, sv, ws, dev))
    # top-k / top-p filtered verification (every request filtered)
    for name, tk_v, tp_v in (("topk50", 50, 1.0), ("topp0.9", 0, 0.9), ("topk50_topp0.9", 50, 0.9)):
        tk_d = torch.full((b.batch,), tk_v, dtype=torch.int32, device=dev)
        tp_d = torch.full((b.batch,), tp_v, dtype=torch.float32, device=dev)
        sv = binding.make_sample_args(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample,
                                      acc, tok, None, None, None, tk_d, tp_d)
        ws.ensure(spx.workspace_size(attn_args, sv))
        out[f"sample_{name}_us"] = timed(sample_call(sv))
        out[f"step_{name}_us"] = timed(lambda: spx.verify_step(attn_args, sv, ws, dev))
    ws.status.bitwise_and_(~spx.DEV_DEGENERATE)
    # selective-speculation support and Algorithm 1
    cws = spx.Workspace.allocate(1 << 20, dev)
    out["draft_confidence_us"] = timed(lambda: spx.draft_confidence(b.draft_logits, b.draft_ids, b.q_indptr, ws=cws))
    out["draft_confidence_bytes"] = b.draft_logits.numel() * b.draft_logits.element_size()
    conf = spx.draft_confidence(b.draft_logits, b.draft_ids, b.q_indptr, ws=cws)[2]
    k_in = torch.tensor(b.k_host, dtype=torch.int32, device=dev)
    k_out = torch.empty_like(k_in)
    n_drop = torch.zeros(1, dtype=torch.int32, device=dev)
    out["select_speculation_us"] = timed(lambda: spx.select_speculation(conf, k_in, 0.3, out=k_out, status=status, n_drop=n_drop))
    big = 16384
    conf_big = torch.rand(big, device=dev)
    k_big = torch.ones(big, dtype=torch.int32, device=dev)
    k_big_out = torch.empty_like(k_big)
    out["select_speculation_16k_us"] = timed(lambda: spx.select_speculation(conf_big, k_big, 0.3, out=k_big_out, status=status, n_drop=n_drop))
    ell = b.seq_lens.to(torch.int32)
    tau = torch.full((b.batch,), 32, dtype=torch.int32, device=dev)
    prec = torch.full((b.batch,), 0.83, dtype=torch.float64, device=dev)
    out["lookahead_memory_us"] = timed(lambda: spx.lookahead_memory(ell, tau, prec, 2, 0.7))
    # LM head (hidden 4096, the workload's vocabulary, one row per target position), fused statistics on;
    # torch's bf16 matmul (cuBLAS) beside it as the library reference
    hid = 4096
    gh = torch.Generator(device=dev).manual_seed(spec.seed + 9)
    H = torch.randn((b.total_q, hid), generator=gh, device=dev).to(torch.bfloat16)
    Wt = (torch.randn((spec.vocab, hid), generator=gh, device=dev) * (3.0 / hid ** 0.5)).to(torch.bfloat16)
    lg = torch.empty((b.total_q, spec.vocab + (-spec.vocab) % 8), dtype=torch.bfloat16, device=dev)
    ts = torch.empty((b.total_q, (spec.vocab + binding.LM_TILE_COLS - 1) // binding.LM_TILE_COLS, 2), dtype=torch.float32, device=dev)
    lm_iters = max(3, min(iters, 20))
    saved, iters = iters, lm_iters
    out["lm_head_us"] = timed(lambda: spx.lm_head(H, Wt, logits=lg, tile_stats=ts, status=status))
    out["lm_head_nostats_us"] = timed(lambda: spx.lm_head(H, Wt, logits=lg, want_stats=False, status=status))
    ref_out = torch.empty((b.total_q, spec.vocab), dtype=torch.bfloat16, device=dev)
    out["cublas_matmul_us"] = timed(lambda: torch.matmul(H, Wt.t(), out=ref_out))
    # sampling half on the LM head's logits: own statistics pass over all rows vs the epilogue's statistics
    if b.draft_logits.stride(0) == lg.stride(0):
        s_plain = binding.make_sample_args(lg, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample, acc, tok,
                                           None, spec.vocab)
        s_fused = binding.make_sample_args(lg, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample, acc, tok,
                                           None, spec.vocab, None, None, None, ts)
        ws.ensure(spx.workspace_size(attn_args, s_plain))
        out["sample_on_lm_logits_us"] = timed(sample_call(s_plain))
        out["sample_with_lm_stats_us"] = timed(sample_call(s_fused))
        out["step_on_lm_logits_us"] = timed(lambda: spx.verify_step(attn_args, s_plain, ws, dev))
        out["step_with_lm_stats_us"] = timed(lambda: spx.verify_step(attn_args, s_fused, ws, dev))
    iters = saved
    flops = 2.0 * b.total_q * hid * spec.vocab
    out["lm_head_tflops"] = flops / (out["lm_head_us"] * 1e-6) / 1e12
    out["cublas_matmul_tflops"] = flops / (out["cublas_matmul_us"] * 1e-6) / 1e12
    out["lm_head_weight_gbs"] = Wt.numel() * 2 / (out["lm_head_us"] * 1e-6) / 1e9
    del H, Wt, lg, ts, ref_out
    if int(ws.status.item()) != 0 or int(status.item()) != 0 or int(cws.status.item()) != 0:
        out["status"] = [int(ws.status.item()), int(status.item()), int(cws.status.item())]
    return out


def run_timeline(args):
    """Where the time of one step goes: every kernel of a timeline build of the library
    (-DSPX_TIMELINE=1: per-CTA %globaltimer stamps, about 1.5 us per step) reports when its CTAs
    started and ended.  Steps are launched back to back in windows; the last step of each window is
    read out, and the median over the windows is printed (us from the first CTA of the step)."""
    import numpy as np
    import paper_2609_34370_b200 as spx
    from paper_2609_34370_b200 import binding, build
    binding.LIB_PATH = build.build_timeline()
    spec = W.CONFIGS[args.workload]
    if args.batch:
        spec = W.scaled(spec, batch=args.batch)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    b = W.generate(spec, device=dev)
    out = torch.empty_like(b.q)
    lse = torch.empty(b.q.shape[:2], dtype=torch.float32, device=dev)
    acc = torch.empty(b.batch, dtype=torch.int32, device=dev)
    tok = torch.empty(b.total_q, dtype=torch.int32, device=dev)
    a = binding.make_attn_args(b.q, b.k_cache, b.v_cache, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                               spec.num_kv_heads, spec.page_size, b.num_pages, out, lse, max_q_len=max(b.k_host) + 1)
    s = binding.make_sample_args(b.target_logits, b.draft_logits, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample, acc, tok)
    ws = spx.Workspace.allocate(spx.workspace_size(a, s), dev)
    for _ in range(max(args.warmup, 3)):
        spx.verify_step(a, s, ws, dev)
    torch.cuda.synchronize()
    names = ["plan", "attention", "combine", "logits statistics", "accept", "residual masses", "residual draw"]
    windows, per_window = 12, max(50, min(args.steps, 500))
    rows = {n: [] for n in names}
    step_us = []
    for _ in range(windows):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(per_window):
            spx.verify_step(a, s, ws, dev)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / per_window
        step_us.append(us)
        tl = spx.debug_timeline().astype(np.int64)
        horizon = tl[:, :, 1].max() - int(us * 1e3) - 3000          # CTAs of the last step only
        spans = {}
        for k, n in enumerate(names):
            st, en = tl[k, :, 0], tl[k, :, 1]
            sel = (en > horizon) & (st > horizon - 200000) & (en >= st)
            spans[n] = (st[sel], en[sel])
        starts = [v[0].min() for v in spans.values() if len(v[0])]
        if not starts:
            continue
        t0 = min(starts)
        for n in names:
            st, en = spans[n]
            if len(st) == 0:
                continue
            st, en = (st - t0) / 1e3, (en - t0) / 1e3
            rows[n].append((len(st), st.min(), np.median(st), st.max(), en.min(), np.median(en), en.max(), np.median(en - st)))
        time.sleep(0.2)
    table = {}
    for n in names:
        if rows[n]:
            m = np.median(np.array(rows[n]), axis=0)
            table[n] = {"ctas": int(m[0]), "first_start_us": round(m[1], 1), "median_start_us": round(m[2], 1),
                        "last_start_us": round(m[3], 1), "first_end_us": round(m[4], 1), "median_end_us": round(m[5], 1),
                        "last_end_us": round(m[6], 1), "median_cta_us": round(m[7], 1)}
    print(json.dumps({"timeline": table, "workload": spec.name, "us_per_step_instrumented": round(float(np.median(step_us)), 2),
                      "windows": windows, "steps_per_window": per_window}))
    print("%-18s %6s %31s %31s %10s" % ("kernel", "CTAs", "starts (first / median / last)", "ends (first / median / last)", "CTA us"),
          file=sys.stderr)
    for n, t in table.items():
        print("%-18s %6d %9.1f %9.1f %9.1f   %9.1f %9.1f %9.1f %10.1f" % (
            n, t["ctas"], t["first_start_us"], t["median_start_us"], t["last_start_us"], t["first_end_us"],
            t["median_end_us"], t["last_end_us"], t["median_cta_us"]), file=sys.stderr)


L2_BYTES = 126 << 20


class StepRunner:
    """One workload resident on the device, ready to be stepped.

    Inputs that are smaller than twice the L2 (the whole tiny workload; the long-context workload's
    17 MB of logits) exist in several copies at different addresses and the steps cycle through them,
    so that no timed step finds its inputs in L2; the other tensors are larger than L2 as they are."""

    def __init__(self, spx, binding, spec, dev, seed):
        self.spx, self.binding, self.spec, self.dev = spx, binding, spec, dev
        b = self.b = W.generate(spec, device=dev, seed=seed)
        self.kv_bytes, self.logit_bytes = b.kv_bytes(), b.logits_bytes()
        self.out = torch.empty_like(b.q)
        self.lse = torch.empty(b.q.shape[:2], dtype=torch.float32, device=dev)
        self.acc = torch.empty(b.batch, dtype=torch.int32, device=dev)
        self.tok = torch.empty(b.total_q, dtype=torch.int32, device=dev)
        kv_sets = 1 if self.kv_bytes >= 2 * L2_BYTES else min(384, -(-2 * L2_BYTES // max(self.kv_bytes, 1)))
        lg_sets = 1 if self.logit_bytes >= 2 * L2_BYTES else min(384, -(-2 * L2_BYTES // max(self.logit_bytes, 1)))
        self.n_sets = max(kv_sets, lg_sets)
        self.keep = []                                             # the copies stay alive
        self.sets = []
        for i in range(self.n_sets):
            kc, vc = (b.k_cache, b.v_cache) if i == 0 or kv_sets == 1 else (b.k_cache.clone(), b.v_cache.clone())
            tl, dl = (b.target_logits, b.draft_logits) if i == 0 or lg_sets == 1 else (b.target_logits.clone(), b.draft_logits.clone())
            self.keep.append((kc, vc, tl, dl))
            a = binding.make_attn_args(b.q, kc, vc, b.kv_strides, b.block_table, b.seq_lens, b.q_indptr,
                                       spec.num_kv_heads, spec.page_size, b.num_pages, self.out, self.lse,
                                       max_q_len=max(b.k_host) + 1)
            sa = binding.make_sample_args(tl, dl, b.draft_ids, b.q_indptr, b.u_accept, b.u_sample, self.acc, self.tok)
            self.sets.append((a, sa))
        self.ws = spx.Workspace.allocate(spx.workspace_size(*self.sets[0]), dev)
        self.rotation = ("inputs larger than L2 (KV + logits re-read from HBM every step)" if self.n_sets == 1 else
                         f"{self.n_sets} input sets cycled ({'KV + ' if kv_sets > 1 else ''}logits copies at distinct addresses, "
                         "more than 2x L2 in total); the rest is larger than L2")
        self.i = 0

    def step(self):
        a, sa = self.sets[self.i % self.n_sets]
        self.i += 1
        self.spx.verify_step(a, sa, self.ws, self.dev)

    def warm(self, n):
        for _ in range(n):
            self.step()
        torch.cuda.synchronize()
        self.launches_per_step = self.spx.last_launch_count()
        self.tokens_per_step = int(self.acc.sum().item()) + self.b.batch
        if int(self.ws.status.item()) != 0:
            raise SystemExit(f"device status {int(self.ws.status.item())} after warm-up ({self.spec.name})")

    def time_steps(self, steps, local, barrier):
        """K whole steps between two CUDA events on the launching stream; clocks sampled meanwhile."""
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        clocks = ClockSampler(local)
        barrier()
        torch.cuda.synchronize()
        clocks.start()
        ev0.record()
        for _ in range(steps):
            self.step()
        ev1.record()
        torch.cuda.synchronize()
        info = clocks.stop()
        barrier()
        return ev0.elapsed_time(ev1), info

    def time_attention(self, n):
        """The verify-attention kernel alone: same launch configuration and inputs, one event pair per
        launch recorded by the library immediately around the kernel (inside the step the sampling
        kernels run beside it on another stream and share its bandwidth)."""
        import ctypes as C
        spx, lib, ws = self.spx, self.spx.load_library(), self.ws
        stream = torch.cuda.current_stream(self.dev).cuda_stream
        events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for e0, e1 in events:
            e0.record()
            e1.record()
        for i in range(3):
            lib.spx_verify_attention(C.byref(self.sets[i % self.n_sets][0]), ws.buf.data_ptr(), ws.buf.numel(),
                                     ws.status.data_ptr(), stream)
        torch.cuda.synchronize()
        for i, (e0, e1) in enumerate(events):
            spx.set_timing_events(e0, e1)
            lib.spx_verify_attention(C.byref(self.sets[i % self.n_sets][0]), ws.buf.data_ptr(), ws.buf.numel(),
                                     ws.status.data_ptr(), stream)
        torch.cuda.synchronize()
        spx.set_timing_events(None, None)
        return [e0.elapsed_time(e1) for e0, e1 in events]


def workload_summary(run: "StepRunner", ms_per_step, attn_ms, clock_info, peak, steps):
    """The per-workload figures of the `workloads` table."""
    attn_avg_ms = sum(attn_ms) / len(attn_ms)
    step_gbs = (run.kv_bytes + run.logit_bytes) / (ms_per_step * 1e-3) / 1e9
    attn_gbs = run.kv_bytes / (attn_avg_ms * 1e-3) / 1e9
    return {"ms_per_step": ms_per_step, "steps": steps, "tokens_per_s": run.tokens_per_step / (ms_per_step * 1e-3),
            "tokens_per_step": run.tokens_per_step, "kv_bytes": run.kv_bytes, "logits_bytes": run.logit_bytes,
            "step_gbs": step_gbs, "step_frac_of_measured": step_gbs / peak,
            "step_frac_of_nominal_8tbs": step_gbs / NOMINAL_HBM_GBS,
            "attn_avg_launch_ms": attn_avg_ms, "attn_gbs": attn_gbs, "attn_frac_of_measured": attn_gbs / peak,
            "attn_traffic_bytes": NCU_TRAFFIC_BYTES.get(run.spec.name), "l2": run.rotation, "clocks": clock_info}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", type=int, default=1, help="index into the five named workloads (default: Llama-3-8B shape)")
    ap.add_argument("--impl", default="spx", choices=["spx", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-others", action="store_true", help="skip the table of the other four workloads (profiling runs)")
    ap.add_argument("--other-steps", type=int, default=300, help="timed steps per workload of the `workloads` table")
    ap.add_argument("--extras", action="store_true",
                    help="also time the pieces around the step: KV append / rollback, verification variants")
    ap.add_argument("--extras-iters", type=int, default=200, help="timed calls per extras entry (profiling runs: a few)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (profiling captures of a smaller case)")
    ap.add_argument("--timeline", action="store_true",
                    help="per-kernel timeline of the step from a timeline build of the library (prints it and exits)")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.steps == 2000:
            args.steps, args.warmup = 3, 1
        run_reference(args)
        return

    import paper_2609_34370_b200 as spx
    from paper_2609_34370_b200 import binding
    if args.timeline:
        run_timeline(args)
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verify step has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    warmup = max(args.warmup, 3)

    def barrier():
        if world > 1:
            dist.barrier()

    peak, peak_kind = measured_peak()
    spec = W.CONFIGS[args.workload]
    if args.batch:
        spec = W.scaled(spec, batch=args.batch, name_suffix=f"-batch{args.batch}")
    run = StepRunner(spx, binding, spec, dev, spec.seed + 1000 * rank)
    b, a, s, ws, acc, tok, out = run.b, run.sets[0][0], run.sets[0][1], run.ws, run.acc, run.tok, run.out
    run.warm(warmup)
    launches_per_step, tokens_per_step = run.launches_per_step, run.tokens_per_step
    ms_total, clock_info = run.time_steps(args.steps, local, barrier)
    attn_ms = run.time_attention(min(args.steps, 200))
    ms_total, job_tokens = reduce_over_ranks(ms_total, tokens_per_step, dev)
    value = job_tokens * args.steps / (ms_total * 1e-3)
    ms_per_step = ms_total / args.steps

    extras = None
    if args.extras and rank == 0:
        extras = time_extras(spx, binding, spec, b, a, dev, iters=args.extras_iters)

    # ---- end to end through the host-buffer entry point (every rank, max time) ----
    b_host = None
    e2e = None
    try:
        if args.no_e2e:
            raise RuntimeError("skipped (--no-e2e)")
        b_host = b.to("cpu")
        pin = {n: getattr(b_host, n).pin_memory() for n in W.VerifyBatch._TENSORS}
        out_h = torch.empty(out.shape, dtype=out.dtype).pin_memory()
        acc_h = torch.empty(acc.shape, dtype=torch.int32).pin_memory()
        tok_h = torch.empty(tok.shape, dtype=torch.int32).pin_memory()
        st_h = torch.zeros(1, dtype=torch.int32).pin_memory()
        ah = binding.make_attn_args(pin["q"], pin["k_cache"], pin["v_cache"], b.kv_strides, pin["block_table"],
                                    pin["seq_lens"], pin["q_indptr"], spec.num_kv_heads, spec.page_size, b.num_pages,
                                    out_h, None, max_q_len=max(b.k_host) + 1)
        sh = binding.make_sample_args(pin["target_logits"], pin["draft_logits"], pin["draft_ids"], pin["q_indptr"],
                                      pin["u_accept"], pin["u_sample"], acc_h, tok_h)
        pool_elems = b.k_cache.numel()
        arena = torch.empty(spx.host_step_arena_size(ah, sh, pool_elems), dtype=torch.uint8, device=dev)
        for _ in range(2):
            spx.verify_step_host(ah, sh, pool_elems, arena, st_h, dev)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(args.e2e_steps):
            spx.verify_step_host(ah, sh, pool_elems, arena, st_h, dev)
        e1.record()
        torch.cuda.synchronize()
        te_ms, _ = reduce_over_ranks(e0.elapsed_time(e1), 0.0, dev)
        assert int(st_h.item()) == 0 and torch.equal(acc_h, acc.cpu()) and torch.equal(tok_h, tok.cpu())
        h2d = sum(pin[n].numel() * pin[n].element_size() for n in W.VerifyBatch._TENSORS)
        d2h = out_h.numel() * out_h.element_size() + acc_h.numel() * 4 + tok_h.numel() * 4 + 4
        e2e = {"value": job_tokens * args.e2e_steps / (te_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps}
        del arena, pin
    except Exception as exc:  # reported, never hidden
        e2e = {"value": None, "unit": UNIT, "error": repr(exc)}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    kv_bytes, logit_bytes = run.kv_bytes, run.logit_bytes
    attn_avg_ms = sum(attn_ms) / len(attn_ms)
    achieved = kv_bytes / (attn_avg_ms * 1e-3) / 1e9
    step_gbs = (kv_bytes + logit_bytes) / (ms_per_step * 1e-3) / 1e9
    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": spec.dtype, "data": "synthetic",
        "config": {"workload": spec.name, "batch": spec.batch, "q_heads": spec.num_q_heads,
                   "kv_heads": spec.num_kv_heads, "head_dim": spec.head_dim, "page_size": spec.page_size,
                   "vocab": spec.vocab, "total_q_rows": b.total_q, "kv_tokens": sum(b.seq_lens_host),
                   "kv_bytes": kv_bytes, "logits_bytes": logit_bytes, "tokens_per_step": tokens_per_step,
                   "l2": run.rotation, "parallelism": "replicas" if world > 1 else "single"},
        "clocks": clock_info,
        "e2e": e2e,
        "gpu_launches": launches_per_step * args.steps,
        "roofline": {"bound": "hbm", "kernel": "verify-attention (timed alone, %d launches)" % len(attn_ms),
                     "achieved": achieved, "peak": peak, "peak_kind": peak_kind + " copy bandwidth",
                     "unit": "GB/s", "frac": achieved / peak, "traffic": NCU_TRAFFIC_BYTES.get(spec.name),
                     "algorithmic_bytes": kv_bytes, "avg_launch_ms": attn_avg_ms},
        "step_hbm": {"bytes": kv_bytes + logit_bytes, "achieved_gbs": step_gbs,
                     "frac_of_measured": step_gbs / peak, "frac_of_nominal_8tbs": step_gbs / NOMINAL_HBM_GBS},
    }
    if extras is not None:
        result["extras"] = extras
    if not args.no_cpu_baseline:
        try:
            n_req = oracle_sample_size(spec)
            bc = b_host if b_host is not None else b.to("cpu")
            dt, otok, threads = time_oracle(bc, n_req)
            passes, total_t, total_tok = 1, dt, otok
            while total_t < 10.0 and passes < 64:         # about 10 s of CPU work
                dt, otok, threads = time_oracle(bc, n_req)
                passes, total_t, total_tok = passes + 1, total_t + dt, total_tok + otok
            result["cpu_baseline"] = {"value": total_tok / total_t, "unit": UNIT, "cores": threads, "kind": "oracle",
                                      "sample": f"first {n_req} of {spec.batch} requests, {passes} passes ({total_t:.1f} s)"}
            result["cpu_baseline"]["sampling_vs_gpu"] = sampling_agreement(bc, n_req, acc, tok)
        except Exception as exc:
            result["cpu_baseline"] = {"value": None, "unit": UNIT, "error": repr(exc), "kind": "oracle"}

    # ---- the other named workloads, same timing, a shorter run each (single-GPU default run only) ----
    if world == 1 and not args.no_others and not args.batch:
        table = {spec.name: workload_summary(run, ms_per_step, attn_ms, clock_info, peak, args.steps)}
        del run, b, a, s, ws, b_host
        torch.cuda.empty_cache()
        for other in W.CONFIGS:
            if other.name in table:
                continue
            try:
                r2 = StepRunner(spx, binding, other, dev, other.seed)
                r2.warm(max(warmup, 10))
                k2 = max(200, args.other_steps)
                ms2, clk2 = r2.time_steps(k2, local, barrier)
                table[other.name] = workload_summary(r2, ms2 / k2, r2.time_attention(min(k2, 200)), clk2, peak, k2)
                del r2
                torch.cuda.empty_cache()
            except Exception as exc:  # reported, never hidden
                table[other.name] = {"error": repr(exc)}
        result["workloads"] = {w.name: table[w.name] for w in W.CONFIGS if w.name in table}
    print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def sampling_agreement(b_cpu, n_req, acc_gpu, tok_gpu):
    """Accepted lengths and emitted tokens of the device path against the oracle's on the sample the
    CPU baseline timed: requests that agree bit for bit / requests compared.  (The tests classify
    the rest into the counted near-tie classes; here they are only counted.)"""
    import oracle
    sb = sub_batch(b_cpu, n_req)
    res = oracle.rejection_sample(sb.target_logits, sb.draft_logits, sb.draft_ids, sb.q_indptr, sb.u_accept, sb.u_sample)
    acc_g, tok_g = acc_gpu.cpu(), tok_gpu.cpu()
    qi = sb.q_indptr.tolist()
    exact = 0
    for r in range(n_req):
        if int(acc_g[r]) == int(res.accepted_len[r]) and torch.equal(tok_g[qi[r]:qi[r + 1]], res.out_tokens[qi[r]:qi[r + 1]]):
            exact += 1
    return {"requests": n_req, "bit_exact": exact}


if __name__ == "__main__":
    main()
