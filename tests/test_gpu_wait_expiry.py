"""The bounded waits of the kernels, on the path where the limit runs out.

Every spin on a barrier in the library (attention roles, the logits ring, the LM head) has a cycle
limit; when it runs out the role raises SPX_DEV_TIMEOUT, sets its CTA's abort flag and returns.  A
wait-test build of the library (limit 100k cycles, about 50 us) carries a one-block kernel in which
each wait helper waits for a signal that never comes: no fault, no unbounded spin, the kernel
returns by itself.  The regular library refuses the call.
"""
import ctypes as C
import time

import pytest
import torch

import spx_workloads as W
import paper_2609_34370_b200 as spx
from paper_2609_34370_b200 import binding, build
from parity_util import check_attention, check_sampling, gpu_attention, gpu_sample, oracle_attention

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_waits_run_out_with_an_error_status_and_the_context_stays_usable():
    lib = C.CDLL(build.build_wait_test())
    lib.spx_debug_wait_expiry.restype = C.c_int
    lib.spx_debug_wait_expiry.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    report = torch.zeros(11, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    assert lib.spx_debug_wait_expiry(report.data_ptr(), status.data_ptr(), None) == binding.OK
    torch.cuda.synchronize()
    elapsed = time.perf_counter() - t0
    rep = report.cpu().tolist()
    assert elapsed < 0.5, elapsed                                  # 100k cycles, not a second
    assert int(status.item()) & spx.DEV_TIMEOUT
    assert rep[0:4] == [2, 2, 2, 2], rep                           # every wait gave up, none was satisfied
    assert rep[8:11] == [1, 1, 1], rep                             # each helper raised its abort flag
    assert 100000 <= rep[4] < 5000000 and 100000 <= rep[6] < 5000000 and 100000 <= rep[7] < 5000000, rep
    assert rep[5] <= rep[4] + 200000, rep                          # the second attention role left with the first
    # the regular library refuses the call and a normal step afterwards is still right
    reg = spx.load_library()
    assert reg.spx_debug_wait_expiry(report.data_ptr(), status.data_ptr(), None) == binding.ERR_UNSUPPORTED
    spec = W.scaled(W.CONFIGS[1], batch=4, ctx_div=8, vocab=5000)
    b_cpu = W.generate(spec)
    b = b_cpu.to(DEV)
    out, lse, ws = gpu_attention(b)
    assert int(ws.status.item()) == 0
    ref_o, ref_l = oracle_attention(b_cpu)
    check_attention(b_cpu, out, lse, ref_o, ref_l)
    acc, tok, _, ws2 = gpu_sample(b)
    assert int(ws2.status.item()) == 0
    assert not check_sampling(b_cpu, acc, tok).hard_mismatch
