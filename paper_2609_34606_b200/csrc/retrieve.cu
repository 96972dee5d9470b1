// Page-level retrieval of the hierarchical KV cache (Section 3.2, Stage 2): a KV page is a run of
// kv_page_blocks consecutive 64-token blocks; its score is
//     alpha_j = mean_h( Qbar_h . Kbar_{j,h} ) * scale
// with the chunk's average query and the page's average key, both taken from sums the selection
// path already keeps (query tile sums, per-block key sums), and the top-K_p pages are kept.
#include <cuda_bf16.h>

#include "hsa_internal.h"

namespace hsa {

namespace {

__device__ __forceinline__ uint32_t rt_order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // ascending with the float order
}

// One CTA per KV page: fp64 dot of the query sum and the page's key sum over all heads and dims.
__global__ void __launch_bounds__(256) kv_page_score_kernel(RetrieveArgs a) {
  __shared__ double red[256];
  const int j = blockIdx.x;
  const int64_t nblk = (a.n_tokens + kBlock - 1) / kBlock;
  const int64_t b0 = static_cast<int64_t>(j) * a.kv_page_blocks;
  const int64_t b1 = min64(nblk, b0 + a.kv_page_blocks);
  const int n_tiles = (a.n_q + kTileM - 1) / kTileM;
  double part = 0.0;
  for (int idx = threadIdx.x; idx < a.H * a.D; idx += 256) {
    const int h = idx / a.D, e = idx % a.D;
    double qs = 0.0;
    for (int t = 0; t < n_tiles; ++t) qs += static_cast<double>(a.qpart[(static_cast<size_t>(t) * a.H + h) * a.D + e]);
    double ks = 0.0;
    for (int64_t b = b0; b < b1; ++b)
      ks += static_cast<double>(a.ksum[(static_cast<size_t>(h) * a.max_pages + b) * a.D + e]);
    part += qs * ks;
  }
  red[threadIdx.x] = part;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (static_cast<int>(threadIdx.x) < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const int64_t toks = min64(a.n_tokens, b1 * kBlock) - b0 * kBlock;
    const double alpha = red[0] / (static_cast<double>(a.n_q) * static_cast<double>(toks) * a.H) *
                         static_cast<double>(a.scale);
    const float f = static_cast<float>(alpha);
    a.keys[j] = rt_order_key(f);
    if (a.scores_out) a.scores_out[j] = f;
  }
}

// One CTA: rank every page by (score descending, id ascending), keep the first top_kp, ascending ids.
__global__ void __launch_bounds__(256) kv_page_topk_kernel(RetrieveArgs a, int n_pages) {
  extern __shared__ uint32_t rkeys[];  // [n_pages] keys, then [n_pages] selected flags
  uint32_t* flag = rkeys + n_pages;
  for (int j = threadIdx.x; j < n_pages; j += 256) rkeys[j] = a.keys[j];
  __syncthreads();
  for (int j = threadIdx.x; j < n_pages; j += 256) {
    const uint32_t kj = rkeys[j];
    int rank = 0;
    for (int i = 0; i < n_pages; ++i) rank += (rkeys[i] > kj) || (rkeys[i] == kj && i < j);
    flag[j] = rank < a.top_kp ? 1u : 0u;
  }
  __syncthreads();
  for (int j = threadIdx.x; j < n_pages; j += 256) {
    if (!flag[j]) continue;
    int pos = 0;
    for (int i = 0; i < j; ++i) pos += static_cast<int>(flag[i]);
    a.page_ids[pos] = j;
  }
}

}  // namespace

cudaError_t launch_retrieve(const RetrieveArgs& a, int n_pages, cudaStream_t st) {
  kv_page_score_kernel<<<n_pages, 256, 0, st>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  kv_page_topk_kernel<<<1, 256, static_cast<size_t>(n_pages) * 8, st>>>(a, n_pages);
  return cudaGetLastError();
}

}  // namespace hsa
