// Intra-chunk part of the causal linear branch.  When the query chunk is the most recently
// appended chunk, query i may only see the chunk's own keys up to its position; the state of
// everything before the chunk is applied by the forward kernel, and this kernel supplies
//   num[i,h,:] = sum_{q_pos0 <= j <= q_pos0+i} (phi(q_i).phi(k_j)) v_j,   den[i,h] = sum of weights
// read from the pool pages.  Plain SIMT: this variant is for the small causal case, not the
// measured path.
#include <cuda_bf16.h>

#include "hsa_internal.h"

namespace hsa {

template <int D>
__global__ void __launch_bounds__(256) causal_linear_kernel(CausalLinArgs a) {
  constexpr int PER = D / 32;
  __shared__ float red_num[8][D];
  __shared__ float red_den[8];
  const int i = blockIdx.x, h = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float fq[PER], num[PER];
  const __nv_bfloat16* qrow =
      a.q + static_cast<size_t>(i) * a.q_ts + static_cast<size_t>(h) * a.q_hs + lane * PER;
#pragma unroll
  for (int e = 0; e < PER; ++e) {
    const float x = __bfloat162float(qrow[e]);
    fq[e] = a.relu ? fmaxf(x, 0.f) : (x > 0.f ? x + 1.f : expf(x));
    num[e] = 0.f;
  }
  float den = 0.f;
  const int64_t j_hi = min64(a.n_tokens - 1, a.q_pos0 + i);
  for (int64_t j = a.q_pos0 + warp; j <= j_hi; j += 8) {
    const int64_t b = j / kBlock;
    const size_t rowi = (static_cast<size_t>(a.page_table[b]) * a.H + h) * kBlock + (j - b * kBlock);
    const __nv_bfloat16* kr = a.k_pool + rowi * D + lane * PER;
    const __nv_bfloat16* vr = a.v_pool + rowi * D + lane * PER;
    float w = 0.f;
#pragma unroll
    for (int e = 0; e < PER; ++e) {
      const float x = __bfloat162float(kr[e]);
      w = fmaf(fq[e], a.relu ? fmaxf(x, 0.f) : (x > 0.f ? x + 1.f : expf(x)), w);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) w += __shfl_xor_sync(0xffffffffu, w, o);
    den += w;
#pragma unroll
    for (int e = 0; e < PER; ++e) num[e] = fmaf(w, __bfloat162float(vr[e]), num[e]);
  }
#pragma unroll
  for (int e = 0; e < PER; ++e) red_num[warp][lane * PER + e] = num[e];
  if (lane == 0) red_den[warp] = den;
  __syncthreads();
  if (threadIdx.x < D) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += red_num[w][threadIdx.x];
    a.lin_num[(static_cast<size_t>(i) * a.H + h) * D + threadIdx.x] = s;
  }
  if (threadIdx.x == 0) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += red_den[w];
    a.lin_den[static_cast<size_t>(i) * a.H + h] = s;
  }
}

cudaError_t launch_causal_linear(const CausalLinArgs& a, cudaStream_t st) {
  dim3 grid(a.n_q, a.H);
  if (a.D == 128)
    causal_linear_kernel<128><<<grid, 256, 0, st>>>(a);
  else
    causal_linear_kernel<64><<<grid, 256, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace hsa
