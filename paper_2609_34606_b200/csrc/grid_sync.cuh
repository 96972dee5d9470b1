// A barrier among the co-resident CTAs of one cooperative launch, kept entirely on the device.
#pragma once
#include <stdint.h>

#include "hsa_internal.h"

namespace hsa {

// bar[0] = arrive count, bar[1] = generation (both zero-initialised once; the count is back at zero
// after every completed barrier).  Exactly n CTAs call this with the same `bar`: each reads the
// generation, arrives, and waits for the generation to change; the last one to arrive puts the
// count back to zero and advances the generation.  Nothing depends on host-side bookkeeping, so a
// launch captured in a CUDA graph behaves the same on every replay.  The wait is bounded (wait_ns):
// on expiry -- or when another CTA has already recorded a timeout -- the status word gets
// HSA_ERR_DEVICE_TIMEOUT and the call returns false.  All threads of the CTA call it; writes made
// by any thread of any arriving CTA before the call are visible to every CTA after it.
__device__ __forceinline__ bool device_barrier(unsigned* bar, unsigned n, int32_t* status, unsigned long long wait_ns) {
  __shared__ int bar_ok;
  __syncthreads();
  if (threadIdx.x == 0) {
    int ok = 1;
    unsigned gen;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(gen) : "l"(bar + 1) : "memory");
    __threadfence();
    const unsigned arrived = atomicAdd(bar, 1u);
    if (arrived == n - 1) {
      bar[0] = 0u;  // ordered before the new generation by the release below
      asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(bar + 1), "r"(gen + 1u) : "memory");
    } else {
      unsigned long long t0 = 0;
      for (unsigned i = 0;; ++i) {
        unsigned v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(bar + 1) : "memory");
        if (v != gen) break;
        if ((i & 63u) == 63u) {
          unsigned long long now;
          asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
          if (t0 == 0) t0 = now;
          // another CTA gave up already, or this one has waited long enough
          if (*reinterpret_cast<volatile int32_t*>(status) == kDevTimeout || now - t0 > wait_ns) {
            atomicCAS(status, 0, kDevTimeout);
            ok = 0;
            break;
          }
        }
      }
    }
    __threadfence();
    bar_ok = ok;
  }
  __syncthreads();
  return bar_ok != 0;
}

}  // namespace hsa
