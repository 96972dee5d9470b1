// Linear branch alone (the "linear only" mode of hsa_forward, head_dim 128):
//   out[i,h] = g_lin * phi(q_i)^T S[h] / (phi(q_i)^T z[h]),   phi(x) = elu(x) + 1
// A lean kernel for the case with no sparse branch: the only traffic is Q in and out out, so it is
// bound by HBM, not by the tensor cores.
// One persistent CTA per SM walks over a contiguous run of (head, query tile) items; the roles form
// a pipeline, so that the load of one tile, the phi(Q) arithmetic of the next, the MMAs of a third
// and the write-out of a fourth overlap:
//   warp 0      (one lane)  TMA loads of the [128 x 128] Q tiles into a three-stage ring
//   warps 2-9   phi(Q) written in place (it is the K-major A operand) + the denominators phi(q).z
//   warp 1      (one lane)  16 tcgen05 MMAs per tile against S_hi and S_lo (kept in shared memory;
//               reloaded by the same lane when the run crosses into the next head) into one of two
//               TMEM accumulators
//   warps 10-17 accumulator -> normalised, gated bf16 rows staged in the tile's ring stage (phi(Q)
//               is dead by then) -> TMA store -> the stage goes back to warp 0
// Every wait is bounded; on expiry the CTA records a timeout and leaves.
#include <cuda_bf16.h>

#include "hsa_internal.h"
#include "ptx.cuh"

namespace hsa {

#ifdef HSA_TIMING
__device__ long long g_lo_timing[256];
#define LO_T(slot)                                                        \
  do {                                                                    \
    if (blockIdx.x == 0 && (threadIdx.x & 31) == 0) {                     \
      long long t_;                                                       \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));               \
      g_lo_timing[(slot)] = t_;                                           \
    }                                                                     \
  } while (0)
#else
#define LO_T(slot) \
  do {             \
  } while (0)
#endif

namespace {

constexpr int kLoStages = 3;                  // Q ring
constexpr int kLoGroup = 256;                 // threads of the phi group and of the epilogue group
constexpr int kLoThreads = 64 + 2 * kLoGroup;
constexpr int kLoTile = 128 * 128 * 2;        // one [128 x 128] bf16 tile = two swizzled slabs
constexpr int kLoHalf = kLoTile / 2;
constexpr int kLoStats = kLoStages * 2 * 128 * 4;  // partial denominators per stage
constexpr int kLoSmem = (2 + kLoStages) * kLoTile + kLoStats + 256 + 1024;
constexpr uint32_t kLoTmemCols = 256;         // two accumulators

struct LoBars {
  uint64_t q_full[kLoStages];     // Q tile landed
  uint64_t q_empty[kLoStages];    // output tile stored: the stage may be refilled
  uint64_t phi_ready[kLoStages];  // phi(Q) written
  uint64_t mma_done[2];           // accumulator final
  uint64_t acc_free[2];           // accumulator read back
  uint64_t s_full;                // state tiles landed
  uint32_t tmem_base;
  volatile int abort_flag;
};

__device__ __forceinline__ bool lo_wait(uint64_t* bar, uint32_t parity, LoBars* bars, int32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  for (uint32_t i = 1; i < (1u << 24); ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 0u && bars->abort_flag) return false;
  }
  bars->abort_flag = 1;
  atomicCAS(status, 0, kDevTimeout);
  return false;
}

__device__ __forceinline__ float lo_phi(float x) {
  float e;  // elu(x) + 1 = max(x, 0) + exp(min(x, 0))
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(fminf(x, 0.f) * 1.4426950408889634f));
  return fmaxf(x, 0.f) + e;
}

}  // namespace

__global__ void __launch_bounds__(kLoThreads, 1)
hsa_linear_only_kernel(FwdParams p, int n_items, const __grid_constant__ CUtensorMap tm_q,
                       const __grid_constant__ CUtensorMap tm_state, const __grid_constant__ CUtensorMap tm_out) {
  constexpr int D = 128;
  extern __shared__ uint8_t lo_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(lo_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* s_state = smem;                 // S_hi | S_lo, MN-major B operands
  uint8_t* s_ring = smem + 2 * kLoTile;    // Q tile -> phi(Q) -> output tile, per stage
  float* stats = reinterpret_cast<float*>(smem + (2 + kLoStages) * kLoTile);  // [stage][half][128]
  LoBars* bars = reinterpret_cast<LoBars*>(smem + (2 + kLoStages) * kLoTile + kLoStats);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp == 0) LO_T(0);
  const int n_tiles = (p.n_q + kTileM - 1) / kTileM;
  // this CTA's run of items (item = head * n_tiles + tile)
  const int i_begin = static_cast<int>(static_cast<int64_t>(blockIdx.x) * n_items / gridDim.x);
  const int i_end = static_cast<int>(static_cast<int64_t>(blockIdx.x + 1) * n_items / gridDim.x);
  const int my_items = i_end - i_begin;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kLoStages; ++s) {
      mbar_init(&bars->q_full[s], 1);
      mbar_init(&bars->q_empty[s], 1);
      mbar_init(&bars->phi_ready[s], kLoGroup);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&bars->mma_done[a], 1);
      mbar_init(&bars->acc_free[a], kLoGroup);
    }
    mbar_init(&bars->s_full, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_state);
    tma_prefetch_desc(&tm_out);
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, kLoTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  if (warp == 0) LO_T(1);

  if (warp == 0) {
    // ------------------------------------------------------------------ Q producer (one lane)
    if (elect_one_sync()) {
      for (int it = 0; it < my_items; ++it) {
        const int s = it % kLoStages;
        if (it >= kLoStages && !lo_wait(&bars->q_empty[s], ((it / kLoStages) - 1) & 1, bars, p.status)) break;
        const int item = i_begin + it, h = item / n_tiles, tile = item % n_tiles;
        mbar_expect_tx(&bars->q_full[s], kLoTile);
        for (int dh = 0; dh < 2; ++dh)
          tma_load_3d(s_ring + s * kLoTile + dh * kLoHalf, &tm_q, &bars->q_full[s], dh * 64, h, tile * kTileM);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (one lane)
    if (elect_one_sync()) {
      constexpr uint32_t kHiSw = desc_hi_sw128(1024);
      constexpr uint32_t idesc = idesc_bf16_f32(128, D, 0, 1);
      int cur_h = -1, s_loads = 0;
      for (int it = 0; it < my_items; ++it) {
        const int s = it % kLoStages, a = it & 1;
        const int h = (i_begin + it) / n_tiles;
        if (h != cur_h) {
          // next head: its state replaces the old one once the MMAs that read the old one are done
          if (it > 0 && !lo_wait(&bars->mma_done[(it - 1) & 1], ((it - 1) >> 1) & 1, bars, p.status)) break;
          mbar_expect_tx(&bars->s_full, 2 * kLoTile);
          for (int hl = 0; hl < 2; ++hl) {
            const int rbase = ((h * 2 + p.use_prev) * 2 + hl) * D;
            for (int kb = 0; kb < 2; ++kb)
              for (int dh = 0; dh < 2; ++dh)
                tma_load_2d(s_state + hl * kLoTile + dh * kLoHalf + kb * (kBlock * 128), &tm_state, &bars->s_full,
                            dh * 64, rbase + kb * 64);
          }
          if (!lo_wait(&bars->s_full, s_loads & 1, bars, p.status)) break;
          ++s_loads;
          cur_h = h;
        }
        if (!lo_wait(&bars->phi_ready[s], (it / kLoStages) & 1, bars, p.status)) break;
        if (it >= 2 && !lo_wait(&bars->acc_free[a], ((it >> 1) - 1) & 1, bars, p.status)) break;
        tc_fence_after();
        const uint32_t a_lo = desc_lo_sw128(smem_u32(s_ring + s * kLoTile), 16);
        for (int hl = 0; hl < 2; ++hl) {
          const uint32_t b_lo = desc_lo_sw128(smem_u32(s_state + hl * kLoTile), kLoHalf);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = ((kk / 4) * kLoHalf + (kk % 4) * 32) >> 4;
            tc_mma_ss_lo(tmem + 128 * a, a_lo + off, b_lo + kk * 128, kHiSw, idesc, (hl > 0 || kk > 0) ? 1u : 0u);
          }
        }
        tc_commit(&bars->mma_done[a]);
        LO_T(16 + it * 8 + 2);
      }
    }
  } else if (warp < 2 + kLoGroup / 32) {
    // ------------------------------------------------------------------ phi(Q) + denominators
    const int t = threadIdx.x - 64;
    const int r = t & 127, half = t >> 7;  // row of the tile, which 64 dims of it
    const int cbase = half * 64;
#pragma unroll 1
    for (int it = 0; it < my_items; ++it) {
      const int s = it % kLoStages;
      const int h = (i_begin + it) / n_tiles;
      if (!lo_wait(&bars->q_full[s], (it / kLoStages) & 1, bars, p.status)) break;
      if (warp == 2) LO_T(16 + it * 8 + 0);
      uint8_t* s_q = s_ring + s * kLoTile;
      const float4* z4 = reinterpret_cast<const float4*>(p.z + static_cast<size_t>(h) * D + cbase);
      // phi of this thread's half row, in place; the partial denominator uses the rounded values
      // (two accumulators: the sum is not one long dependent chain)
      float den0 = 0.f, den1 = 0.f;
#pragma unroll
      for (int c16 = 0; c16 < 8; ++c16) {
        const float4 za = z4[c16 * 2], zb = z4[c16 * 2 + 1];
        const float z[8] = {za.x, za.y, za.z, za.w, zb.x, zb.y, zb.z, zb.w};
        const int cc = cbase / 8 + c16;  // 16-byte chunk of the row
        uint4* cell = reinterpret_cast<uint4*>(s_q + (cc >> 3) * kLoHalf + r * 128 + (((cc & 7) ^ (r & 7)) << 4));
        const uint4 raw = *cell;
        const uint32_t* qw = reinterpret_cast<const uint32_t*>(&raw);
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float a0 = lo_phi(__uint_as_float(qw[i] << 16));
          const float a1 = lo_phi(__uint_as_float(qw[i] & 0xffff0000u));
          o[i] = pack_bf16(a0, a1);
          den0 = fmaf(__uint_as_float(o[i] << 16), z[2 * i], den0);
          den1 = fmaf(__uint_as_float(o[i] & 0xffff0000u), z[2 * i + 1], den1);
        }
        *cell = make_uint4(o[0], o[1], o[2], o[3]);
      }
      stats[(s * 2 + half) * 128 + r] = den0 + den1;
      fence_proxy_async_smem();  // generic-proxy writes above -> visible to the tensor cores
      mbar_arrive(&bars->phi_ready[s]);  // (release: the epilogue group reads stats after the MMAs)
      if (warp == 2) LO_T(16 + it * 8 + 1);
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int e = threadIdx.x - 64 - kLoGroup;
    const int quad = warp & 3;                         // TMEM lane quadrant of this warp
    const int half = (warp - (2 + kLoGroup / 32)) >> 2;  // which 64 dims of the row
    const int r = quad * 32 + lane;
    const int cbase = half * 64;
    const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
    const bool sig = p.gate_act == 1;
    bool ok = true;
#pragma unroll 1
    for (int it = 0; it < my_items && ok; ++it) {
      const int s = it % kLoStages, a = it & 1;
      const int item = i_begin + it, h = item / n_tiles, tile = item % n_tiles;
      const int row0 = tile * kTileM, row = row0 + r;
      uint8_t* s_q = s_ring + s * kLoTile;
      ok = lo_wait(&bars->mma_done[a], (it >> 1) & 1, bars, p.status);
      if (!ok) break;
      if (warp == 10) LO_T(16 + it * 8 + 3);
      tc_fence_after();
      float den = stats[(s * 2) * 128 + r] + stats[(s * 2 + 1) * 128 + r];
      const bool wr = row < p.n_q;  // rows past the end of the chunk compute but never store
      const float* lnum = nullptr;
      if (wr && p.lin_num != nullptr) {
        lnum = p.lin_num + (static_cast<size_t>(row) * p.H + h) * D;
        den += p.lin_den[static_cast<size_t>(row) * p.H + h];
      }
      const float inv_den = den > 0.f ? 1.f / den : 0.f;
      const __nv_bfloat16* gl =
          (wr && p.g_lin) ? p.g_lin + static_cast<size_t>(row) * p.g_ts + static_cast<size_t>(h) * p.g_hs : nullptr;
      const int g_ds = static_cast<int>(p.g_ds);
#pragma unroll 1
      for (int c0 = cbase; c0 < cbase + 64; c0 += 32) {
        uint32_t acc[32];
        tmem_ld32(tmem + lane_off + 128 * a + c0, acc);
        tc_wait_ld();
        if (c0 + 32 == cbase + 64) {  // last read of the accumulator: the MMAs of tile it + 2 may have it
          tc_fence_before();
          mbar_arrive(&bars->acc_free[a]);
        }
        uint32_t packed[16];
        if (gl == nullptr && lnum == nullptr) {
#pragma unroll
          for (int i = 0; i < 32; i += 2)
            packed[i >> 1] = pack_bf16(__uint_as_float(acc[i]) * inv_den, __uint_as_float(acc[i + 1]) * inv_den);
        } else {
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            float w0 = inv_den, w1 = inv_den, l0 = 0.f, l1 = 0.f;
            if (gl) {
              const float g0 = __bfloat162float(gl[(c0 + i) * g_ds]), g1 = __bfloat162float(gl[(c0 + i + 1) * g_ds]);
              w0 *= sig ? __fdividef(1.f, 1.f + __expf(-g0)) : g0;
              w1 *= sig ? __fdividef(1.f, 1.f + __expf(-g1)) : g1;
            }
            if (lnum) {
              l0 = lnum[c0 + i];
              l1 = lnum[c0 + i + 1];
            }
            packed[i >> 1] = pack_bf16(w0 * (__uint_as_float(acc[i]) + l0), w1 * (__uint_as_float(acc[i + 1]) + l1));
          }
        }
        // the phi(Q) tile is dead: the output row goes where it was, in the swizzled layout the
        // output tensor map expects
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          const int cc = (c0 >> 3) + q4;
          *reinterpret_cast<uint4*>(s_q + (cc >> 3) * kLoHalf + r * 128 + (((cc & 7) ^ (r & 7)) << 4)) =
              make_uint4(packed[4 * q4], packed[4 * q4 + 1], packed[4 * q4 + 2], packed[4 * q4 + 3]);
        }
      }
      if (warp == 10) LO_T(16 + it * 8 + 4);
      fence_proxy_async_smem();
      asm volatile("bar.sync 1, %0;" ::"n"(kLoGroup) : "memory");
      if (e == 0) {
        for (int dh = 0; dh < 2; ++dh) tma_store_3d(&tm_out, s_q + dh * kLoHalf, dh * 64, h, row0);
        tma_store_commit();
        tma_store_wait_read();  // the tile must stay put until it has been read
        mbar_arrive(&bars->q_empty[s]);
        LO_T(16 + it * 8 + 5);
      }
    }
    if (e == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (warp == 10) LO_T(2);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kLoTmemCols);
  }
}

#ifdef HSA_TIMING
extern "C" int hsa_debug_read_lo_timing(long long* host_out, int n) {
  return static_cast<int>(cudaMemcpyFromSymbol(host_out, g_lo_timing, sizeof(long long) * n));
}
#endif

cudaError_t linear_only_init() {
  return cudaFuncSetAttribute(hsa_linear_only_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kLoSmem);
}

cudaError_t launch_linear_only(const FwdParams& p, int nsm, const CUtensorMap& tm_q, const CUtensorMap& tm_state,
                               const CUtensorMap& tm_out, cudaStream_t st) {
  const int n_tiles = (p.n_q + kTileM - 1) / kTileM;
  const int n_items = n_tiles * p.H;
  const int grid = n_items < nsm ? n_items : nsm;  // one persistent CTA per SM
  hsa_linear_only_kernel<<<grid, kLoThreads, kLoSmem, st>>>(p, n_items, tm_q, tm_state, tm_out);
  return cudaGetLastError();
}

}  // namespace hsa
