// Self-test of the bounded wait: one thread waits on a barrier that nobody will ever complete,
// gives up after `spins` polls and reports AIBX_ERR_TIMEOUT like the copy kernels do.  Nothing
// is in flight, so the context stays fully usable afterwards.
#pragma once

#include "aibx_common.cuh"
#include "kv_copy.cuh"

namespace aibx {

__global__ void bounded_wait_probe_kernel(unsigned int spins) {
  __shared__ __align__(8) unsigned long long s_bar;
  if (threadIdx.x != 0) return;
  mbar_init(smem_u32(&s_bar), 1u);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  unsigned int n = 0;
  while (!mbar_try_wait(smem_u32(&s_bar), 0u)) {
    if (++n >= spins) {
      raise_status(AIBX_ERR_TIMEOUT);
      return;
    }
  }
}

}  // namespace aibx
