// Wait-test builds only (-DSPX_WAIT_TEST=1 with a small -DSPX_WAIT_LIMIT_CYCLES): one tiny kernel
// in which each bounded-wait helper of the library waits on a barrier that nothing ever arrives at.
// Nothing faults and nothing spins without a limit: every wait ends by its cycle limit or by the
// abort flag another role raised, the kernel returns, and the host reads what happened.
#pragma once
#include "attn_tc.cuh"
#include "lm_head.cuh"
#include "sampler.cuh"

namespace spx {

// report[i]: 1 = the wait of role i returned true (must not happen), 2 = it gave up;
// report[4 + i]: clock cycles role i spent waiting.  Roles: 0 attention barrier wait (expires),
// 1 a second attention role on another barrier of the same CTA (leaves by the abort flag or its
// own limit), 2 the logits ring's wait, 3 the LM head's wait.
__global__ void __launch_bounds__(128) wait_expiry_kernel(int32_t *report, int32_t *dev_status) {
  __shared__ TcBarriers bars;
  __shared__ LmBarriers lbars;
  __shared__ uint64_t ring_bar;
  __shared__ int ring_abort;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bars.k_full[0], 1);
    tc::mbar_init(&bars.v_full[0], 1);
    tc::mbar_init(&lbars.full[0], 1);
    tc::mbar_init(&ring_bar, 1);
    bars.abort = 0;
    lbars.abort = 0;
    ring_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const int role = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) {
    const long long t0 = clock64();
    bool got = false;
    if (role == 0) got = tc::mbar_wait(&bars.k_full[0], 0, &bars, dev_status);
    else if (role == 1) got = tc::mbar_wait(&bars.v_full[0], 0, &bars, dev_status);
    else if (role == 2) got = ring_wait(&ring_bar, 0, &ring_abort, dev_status);
    else got = lm_wait(&lbars.full[0], 0, &lbars, dev_status);
    report[role] = got ? 1 : 2;
    report[4 + role] = (int32_t)min(clock64() - t0, (long long)0x7fffffff);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    report[8] = bars.abort;
    report[9] = lbars.abort;
    report[10] = ring_abort;
  }
}

}  // namespace spx
