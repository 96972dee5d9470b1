// A barrier among the co-resident CTAs of one cooperative launch, kept entirely on the device.
#pragma once
#include <stdint.h>

#include "hsa_internal.h"

namespace hsa {

// bar[0] = arrive count, bar[1] = generation: one 8-byte word (both halves zero-initialised once; the
// count is back at zero after every completed barrier).  Exactly n CTAs call this with the same
// `bar`: each arrives with ONE 64-bit atomic add, which also hands it the generation it arrived in,
// and waits for the generation to change; the last one to arrive puts the count back to zero and
// advances the generation, again in one step.  Nothing depends on host-side bookkeeping, so a
// launch captured in a CUDA graph behaves the same on every replay.  The wait is bounded (wait_ns):
// on expiry -- or when another CTA has already recorded a timeout -- the status word gets
// HSA_ERR_DEVICE_TIMEOUT and the call returns false.  All threads of the CTA call it; writes made
// by any thread of any arriving CTA before the call are visible to every CTA after it.
__device__ __forceinline__ bool device_barrier(unsigned* bar, unsigned n, int32_t* status, unsigned long long wait_ns) {
  __shared__ int bar_ok;
  __syncthreads();
  if (threadIdx.x == 0) {
    int ok = 1;
    unsigned long long* word = reinterpret_cast<unsigned long long*>(bar);  // 8-byte aligned
    __threadfence();
    const unsigned long long old = atomicAdd(word, 1ull);
    const unsigned gen = static_cast<unsigned>(old >> 32);
    if (static_cast<unsigned>(old) == n - 1) {
      __threadfence();  // the other CTAs' writes, seen through their arrivals, go on to the waiters
      atomicAdd(word, (1ull << 32) - static_cast<unsigned long long>(n));  // count -> 0, generation + 1
    } else {
      unsigned long long t0 = 0;
      for (unsigned i = 0;; ++i) {
        unsigned long long v;
        asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(word) : "memory");
        if (static_cast<unsigned>(v >> 32) != gen) break;
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
