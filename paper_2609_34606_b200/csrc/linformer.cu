// Linformer form of the linear branch (Section 3.3 "Linear branch", Eq. 3; Appendix G):
// per appended segment of L tokens and per head, K~ = E_K^T K and V~ = E_V^T V (r rows each) are
// appended to a compressed pool that has the page layout of the main pool, so that the forward
// kernel can run plain softmax attention over it ("every block selected").
//
// One CTA computes a [128 rows of r] x [128 dims] tile of K~ or V~ for one head:
//   C (fp32 in TMEM) = sum over token blocks of  E[tokens, 128 r]^T  X[tokens, 128 d]
// with both operands staged in shared memory in the 128-byte-swizzled MN-major layout (tcgen05,
// K = tokens), double-buffered against the next block's loads, and writes bf16 rows to the pool.
#include <cuda_bf16.h>

#include "hsa_internal.h"
#include "ptx.cuh"

namespace hsa {

namespace {

constexpr int kLcThreads = 512;
constexpr int kLcRowGroups = kLcThreads / 16;
constexpr int kLcRows = kBlock / kLcRowGroups;  // 2 token rows per thread and block
constexpr int kLcTile = 64 * 128 * 2;
constexpr int kLcStage = 2 * kLcTile;  // E tile | X tile
constexpr int kLcSmem = 2 * kLcStage + 64 + 1024;

struct LcBars {
  uint64_t mma_done[2];
  uint64_t all_done;
  uint32_t tmem_base;
  volatile int abort_flag;
};

__device__ __forceinline__ bool lc_wait(uint64_t* bar, uint32_t parity, LcBars* bars, int32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  for (uint32_t i = 1; i < (1u << 24); ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 0u && bars->abort_flag) return false;
  }
  bars->abort_flag = 1;
  atomicCAS(status, 0, kDevTimeout);
  return false;
}

}  // namespace

__global__ void __launch_bounds__(kLcThreads, 1) linformer_compress_kernel(LinformerArgs a) {
  constexpr int D = 128;
  extern __shared__ uint8_t lc_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(lc_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  LcBars* bars = reinterpret_cast<LcBars*>(smem + 2 * kLcStage);
  const int h = blockIdx.y;
  const int rtiles = a.rank / 128;
  const int which = blockIdx.x / rtiles;  // 0: keys, 1: values
  const int rt = blockIdx.x % rtiles;
  const __nv_bfloat16* E = (which == 0 ? a.e_k : a.e_v) + static_cast<size_t>(h) * a.seg_tokens * a.rank + rt * 128;
  const __nv_bfloat16* X = (which == 0 ? a.k : a.v) + static_cast<size_t>(h) * a.head_stride;
  __nv_bfloat16* pool = which == 0 ? a.kc_pool : a.vc_pool;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ch = threadIdx.x & 15, rg = threadIdx.x >> 4;
  const int nblk = (a.seg_tokens + kBlock - 1) / kBlock;

  if (threadIdx.x == 0) {
    mbar_init(&bars->mma_done[0], 1);
    mbar_init(&bars->mma_done[1], 1);
    mbar_init(&bars->all_done, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
    if (blockIdx.x == 0) a.ccnt[h] = (a.seg_index + 1) * (a.rank / kBlock);  // compressed pages now valid
  }
  if (warp == 0) {
    tmem_alloc(&bars->tmem_base, 128);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  uint4 ereg[kLcRows], xreg[kLcRows];
  auto load_block = [&](int bi, uint4 (&ee)[kLcRows], uint4 (&xx)[kLcRows]) {
#pragma unroll
    for (int i = 0; i < kLcRows; ++i) {
      const int t = bi * kBlock + rg + kLcRowGroups * i;
      if (t < a.seg_tokens) {
        ee[i] = *reinterpret_cast<const uint4*>(E + static_cast<size_t>(t) * a.rank + ch * 8);
        xx[i] = *reinterpret_cast<const uint4*>(X + static_cast<size_t>(t) * a.tok_stride + ch * 8);
      } else {  // rows past the end of the segment contribute nothing
        ee[i] = make_uint4(0, 0, 0, 0);
        xx[i] = make_uint4(0, 0, 0, 0);
      }
    }
  };
  load_block(0, ereg, xreg);
  bool ok = true;
#pragma unroll 1
  for (int bi = 0; bi < nblk; ++bi) {
    const int stage = bi & 1;
    uint8_t* st_e = smem + stage * kLcStage;
    uint8_t* st_x = st_e + kLcTile;
    uint4 enext[kLcRows], xnext[kLcRows];
    if (bi + 1 < nblk) load_block(bi + 1, enext, xnext);
    if (bi >= 2) ok = lc_wait(&bars->mma_done[stage], ((bi >> 1) - 1) & 1, bars, a.status) && ok;
#pragma unroll
    for (int i = 0; i < kLcRows; ++i) {
      const int r = rg + kLcRowGroups * i;
      const uint32_t soff = (ch >> 3) * (kLcTile / 2) + r * 128 + (((ch & 7) ^ (r & 7)) << 4);
      *reinterpret_cast<uint4*>(st_e + soff) = ereg[i];
      *reinterpret_cast<uint4*>(st_x + soff) = xreg[i];
    }
    fence_proxy_async_smem();
    __syncthreads();
    if (warp == 0) {
      if (elect_one_sync() && ok) {
        tc_fence_after();
        constexpr uint32_t idesc = idesc_bf16_f32(128, 128, 1, 1);
        constexpr uint32_t hi = desc_hi_sw128(1024);
        const uint32_t a_lo = desc_lo_sw128(smem_u32(st_e), kLcTile / 2);
        const uint32_t b_lo = desc_lo_sw128(smem_u32(st_x), kLcTile / 2);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_ss_lo(tmem, a_lo + kk * 128, b_lo + kk * 128, hi, idesc, (bi > 0 || kk > 0) ? 1u : 0u);
        tc_commit(&bars->mma_done[stage]);
      }
    }
#pragma unroll
    for (int i = 0; i < kLcRows; ++i) {
      ereg[i] = enext[i];
      xreg[i] = xnext[i];
    }
  }
  if (warp == 0) {
    if (elect_one_sync()) tc_commit(&bars->all_done);
  }
  ok = lc_wait(&bars->all_done, 0, bars, a.status) && ok;
  tc_fence_after();
  {
    const int quad = warp & 3, part = warp >> 2;
    const int rr = rt * 128 + quad * 32 + lane;  // row of the compressed segment
    uint32_t v[32];
    tmem_ld32(tmem + (static_cast<uint32_t>(quad * 32) << 16) + part * 32, v);
    tc_wait_ld();
    const int page = a.seg_index * (a.rank / kBlock) + rr / kBlock;
    __nv_bfloat16* dst = pool + ((static_cast<size_t>(page) * a.H + h) * kBlock + (rr % kBlock)) * D + part * 32;
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) pk[i] = pack_bf16(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
#pragma unroll
    for (int i = 0; i < 4; ++i)
      reinterpret_cast<uint4*>(dst)[i] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, 128);
  }
}

cudaError_t linformer_init() {
  return cudaFuncSetAttribute(linformer_compress_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kLcSmem);
}

cudaError_t launch_linformer_compress(const LinformerArgs& a, cudaStream_t st) {
  dim3 grid(2 * (a.rank / 128), a.H);
  linformer_compress_kernel<<<grid, kLcThreads, kLcSmem, st>>>(a);
  return cudaGetLastError();
}

}  // namespace hsa
