// Linformer form of the linear branch (Section 3.3 "Linear branch", Eq. 3; Appendix G):
// per appended segment of L tokens and per head, K~ = E_K^T K and V~ = E_V^T V (r rows each) are
// appended to a compressed pool that has the page layout of the main pool, so that the forward
// kernel can run plain softmax attention over it ("every block selected").
//
// One CTA computes a [128 rows of r] x [128 dims] tile of K~ or V~ for one head:
//   C (fp32 in TMEM) = sum over token blocks of  E[tokens, 128 r]^T  X[tokens, 128 d]
// One lane brings the [64 tokens x 128] tiles of E and of X into a four-stage ring by TMA (both land
// in the 128-byte-swizzled MN-major layout the tensor cores take as they are; rows past the end of
// the segment arrive as zeros), one lane issues four tcgen05 MMAs per block (K = tokens) and hands the
// stage back, and at the end all warps write the bf16 rows to the compressed pool.
#include <cuda_bf16.h>

#include "hsa_internal.h"
#include "ptx.cuh"

namespace hsa {

namespace {

constexpr int kLcThreads = 512;
constexpr int kLcDepth = 4;
constexpr int kLcTile = 64 * 128 * 2;
constexpr int kLcStage = 2 * kLcTile;  // E tile | X tile
constexpr int kLcSmem = kLcDepth * kLcStage + 256 + 1024;

struct LcBars {
  uint64_t full[kLcDepth];
  uint64_t empty[kLcDepth];
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

__global__ void __launch_bounds__(kLcThreads, 1)
linformer_compress_kernel(LinformerArgs a, const __grid_constant__ CUtensorMap tm_ek, const __grid_constant__ CUtensorMap tm_ev,
                          const __grid_constant__ CUtensorMap tm_kin, const __grid_constant__ CUtensorMap tm_vin) {
  constexpr int D = 128;
  extern __shared__ uint8_t lc_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(lc_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  LcBars* bars = reinterpret_cast<LcBars*>(smem + kLcDepth * kLcStage);
  const int h = blockIdx.y;
  const int rtiles = (a.rank + 127) / 128;  // (the last tile may hold 64 rows only: E reads as zeros beyond the rank)
  const int which = blockIdx.x / rtiles;  // 0: keys, 1: values
  const int rt = blockIdx.x % rtiles;
  const CUtensorMap* tm_e = which == 0 ? &tm_ek : &tm_ev;  // [H][seg_tokens][rank], box 64 r x 64 tokens
  const CUtensorMap* tm_x = which == 0 ? &tm_kin : &tm_vin;  // [tokens][H][d], box 64 d x 1 x 64 tokens
  __nv_bfloat16* pool = which == 0 ? a.kc_pool : a.vc_pool;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nblk = (a.seg_tokens + kBlock - 1) / kBlock;
  // the page-write kernel of the same append is launched behind this one as a programmatic
  // dependent and may run beside it (it touches none of this kernel's outputs)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (threadIdx.x == 0) {
    for (int s = 0; s < kLcDepth; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
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

  if (warp == 1) {
    // ------------------------------------------------------------------ producer (one lane)
    if (elect_one_sync()) {
      for (int bi = 0; bi < nblk; ++bi) {
        const int s = bi % kLcDepth;
        if (bi >= kLcDepth && !lc_wait(&bars->empty[s], ((bi / kLcDepth) - 1) & 1, bars, a.status)) break;
        uint8_t* st_e = smem + s * kLcStage;
        uint8_t* st_x = st_e + kLcTile;
        mbar_expect_tx(&bars->full[s], kLcStage);
        for (int half = 0; half < 2; ++half) {
          tma_load_3d(st_e + half * (kLcTile / 2), tm_e, &bars->full[s], rt * 128 + half * 64, bi * kBlock, h);
          tma_load_3d(st_x + half * (kLcTile / 2), tm_x, &bars->full[s], half * 64, h, bi * kBlock);
        }
      }
    }
  } else if (warp == 0) {
    // ------------------------------------------------------------------ MMA issuer (one lane)
    if (elect_one_sync()) {
      constexpr uint32_t idesc = idesc_bf16_f32(128, 128, 1, 1);
      constexpr uint32_t hi = desc_hi_sw128(1024);
      bool ok = true;
      for (int bi = 0; bi < nblk && ok; ++bi) {
        const int s = bi % kLcDepth;
        ok = lc_wait(&bars->full[s], (bi / kLcDepth) & 1, bars, a.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_lo = desc_lo_sw128(smem_u32(smem + s * kLcStage), kLcTile / 2);
        const uint32_t b_lo = desc_lo_sw128(smem_u32(smem + s * kLcStage + kLcTile), kLcTile / 2);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_ss_lo(tmem, a_lo + kk * 128, b_lo + kk * 128, hi, idesc, (bi > 0 || kk > 0) ? 1u : 0u);
        tc_commit(&bars->empty[s]);
      }
      tc_commit(&bars->all_done);
    }
  }
  __syncwarp();
  const bool ok = lc_wait(&bars->all_done, 0, bars, a.status);
  tc_fence_after();
  const int rr = rt * 128 + (warp & 3) * 32 + lane;  // row of the compressed segment
  if (ok && rr < a.rank) {                            // (warp-uniform: the rank is a multiple of 64)
    const int quad = warp & 3, part = warp >> 2;
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

cudaError_t launch_linformer_compress(const LinformerArgs& a, const CUtensorMap& tm_ek, const CUtensorMap& tm_ev,
                                      const CUtensorMap& tm_kin, const CUtensorMap& tm_vin, cudaStream_t st) {
  dim3 grid(2 * ((a.rank + 127) / 128), a.H);
  linformer_compress_kernel<<<grid, kLcThreads, kLcSmem, st>>>(a, tm_ek, tm_ev, tm_kin, tm_vin);
  return cudaGetLastError();
}

}  // namespace hsa
