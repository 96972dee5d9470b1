// Linear branch alone (the "linear only" mode of hsa_forward, head_dim 128):
//   out[i,h] = g_lin * phi(q_i)^T S[h] / (phi(q_i)^T z[h]),   phi(x) = elu(x) + 1
// A lean kernel for the case with no sparse branch: the only traffic is Q in and out out, so it is
// bound by HBM, not by the tensor cores.
// grid (splits, H); a CTA keeps its head's state (bf16 hi + lo halves, 64 KB) in shared memory and
// walks over a run of query tiles.  Per tile: TMA load of the [128 x 128] Q tile, phi(Q) written in
// place (it is the K-major A operand), 16 tcgen05 MMAs against S_hi and S_lo into TMEM, then the
// normalised rows go back through the same shared memory tile to a TMA store.  Two CTAs share an
// SM, so one CTA's loads and stores hide under the other's arithmetic.
#include <cuda_bf16.h>

#include "hsa_internal.h"
#include "ptx.cuh"

namespace hsa {

#ifdef HSA_TIMING
__device__ long long g_lo_timing[256];
#define LO_T(slot)                                                                  \
  do {                                                                              \
    if (blockIdx.x == 0 && blockIdx.y == 0 && (threadIdx.x & 31) == 0) {            \
      long long t_;                                                                 \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                         \
      g_lo_timing[(slot)] = t_;                                                     \
    }                                                                               \
  } while (0)
#else
#define LO_T(slot) \
  do {             \
  } while (0)
#endif

namespace {

constexpr int kLoCompute = 256;               // compute threads (warps 2..9): two per query row
constexpr int kLoThreads = 64 + kLoCompute;   // + TMA warp + MMA warp
constexpr int kLoTile = 128 * 128 * 2;        // one [128 x 128] bf16 tile = two swizzled slabs
constexpr int kLoHalf = kLoTile / 2;
constexpr int kLoStats = 2 * 128 * 4;         // partial denominators
constexpr int kLoSmem = 3 * kLoTile + kLoStats + 256 + 1024;
constexpr uint32_t kLoTmemCols = 128;

struct LoBars {
  uint64_t s_full;     // state landed (once)
  uint64_t q_full;     // Q tile landed
  uint64_t phi_ready;  // phi(Q) written
  uint64_t mma_done;   // accumulator final
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

__global__ void __launch_bounds__(kLoThreads, 2)
hsa_linear_only_kernel(FwdParams p, int tiles_per_cta, const __grid_constant__ CUtensorMap tm_q,
                       const __grid_constant__ CUtensorMap tm_state, const __grid_constant__ CUtensorMap tm_out) {
  constexpr int D = 128;
  extern __shared__ uint8_t lo_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(lo_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* s_state = smem;               // S_hi | S_lo, MN-major B operands
  uint8_t* s_q = smem + 2 * kLoTile;     // Q tile -> phi(Q) -> output tile
  float* stats = reinterpret_cast<float*>(smem + 3 * kLoTile);
  LoBars* bars = reinterpret_cast<LoBars*>(smem + 3 * kLoTile + kLoStats);

  const int h = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp == 0) LO_T(0);
  const int n_tiles = (p.n_q + kTileM - 1) / kTileM;
  const int t_begin = blockIdx.x * tiles_per_cta;
  const int t_end = min(n_tiles, t_begin + tiles_per_cta);
  const int my_tiles = max(0, t_end - t_begin);

  auto load_q = [&](int tile) {
    mbar_expect_tx(&bars->q_full, kLoTile);
    for (int dh = 0; dh < 2; ++dh)
      tma_load_3d(s_q + dh * kLoHalf, &tm_q, &bars->q_full, dh * 64, h, tile * kTileM);
  };
  if (threadIdx.x == 0) {
    mbar_init(&bars->s_full, 1);
    mbar_init(&bars->q_full, 1);
    mbar_init(&bars->phi_ready, kLoCompute);
    mbar_init(&bars->mma_done, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
    if (my_tiles > 0) {
      load_q(t_begin);
      mbar_expect_tx(&bars->s_full, 2 * kLoTile);
      for (int hl = 0; hl < 2; ++hl) {
        const int rbase = ((h * 2 + p.use_prev) * 2 + hl) * D;
        for (int kb = 0; kb < 2; ++kb)
          for (int dh = 0; dh < 2; ++dh)
            tma_load_2d(s_state + hl * kLoTile + dh * kLoHalf + kb * (kBlock * 128), &tm_state, &bars->s_full,
                        dh * 64, rbase + kb * 64);
      }
    }
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

  if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (one lane)
    if (elect_one_sync() && my_tiles > 0) {
      constexpr uint32_t kHiSw = desc_hi_sw128(1024);
      constexpr uint32_t idesc = idesc_bf16_f32(128, D, 0, 1);
      const uint32_t a_lo = desc_lo_sw128(smem_u32(s_q), 16);
      bool ok = lo_wait(&bars->s_full, 0, bars, p.status);
      LO_T(2);
      for (int it = 0; it < my_tiles && ok; ++it) {
        ok = lo_wait(&bars->phi_ready, it & 1, bars, p.status);
        if (!ok) break;
        tc_fence_after();
        for (int hl = 0; hl < 2; ++hl) {
          const uint32_t b_lo = desc_lo_sw128(smem_u32(s_state + hl * kLoTile), kLoHalf);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = ((kk / 4) * kLoHalf + (kk % 4) * 32) >> 4;
            tc_mma_ss_lo(tmem, a_lo + off, b_lo + kk * 128, kHiSw, idesc, (hl > 0 || kk > 0) ? 1u : 0u);
          }
        }
        tc_commit(&bars->mma_done);
        LO_T(32 + it * 8 + 7);
      }
    }
  } else if (warp >= 2) {
    // ------------------------------------------------------------------ phi(Q), epilogue
    const int cw = threadIdx.x - 64;
    const int quad = warp & 3;            // TMEM lane quadrant of this warp
    const int half = (warp - 2) >> 2;     // which 64 dims of the row
    const int r = quad * 32 + lane;       // row inside the tile
    const int cbase = half * 64;
    const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
    const float4* z4 = reinterpret_cast<const float4*>(p.z + static_cast<size_t>(h) * D + cbase);
    const bool sig = p.gate_act == 1;
    bool ok = true;
#pragma unroll 1
    for (int it = 0; it < my_tiles && ok; ++it) {
      const int row0 = (t_begin + it) * kTileM;
      const int row = row0 + r;
      ok = lo_wait(&bars->q_full, it & 1, bars, p.status);
      if (!ok) break;
      if (warp == 2) LO_T(32 + it * 8 + 0);
      // phi of this thread's half row, in place; the partial denominator uses the rounded values
      float den_part = 0.f;
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
          den_part = fmaf(__uint_as_float(o[i] << 16), z[2 * i], den_part);
          den_part = fmaf(__uint_as_float(o[i] & 0xffff0000u), z[2 * i + 1], den_part);
        }
        *cell = make_uint4(o[0], o[1], o[2], o[3]);
      }
      stats[half * 128 + r] = den_part;
      fence_proxy_async_smem();  // generic-proxy writes above -> visible to the tensor cores
      mbar_arrive(&bars->phi_ready);
      if (warp == 2) LO_T(32 + it * 8 + 1);
      asm volatile("bar.sync 1, %0;" ::"n"(kLoCompute) : "memory");
      float den = stats[r] + stats[128 + r];

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

      ok = lo_wait(&bars->mma_done, it & 1, bars, p.status);
      if (!ok) break;
      if (warp == 2) LO_T(32 + it * 8 + 2);
      tc_fence_after();
#pragma unroll 1
      for (int c0 = cbase; c0 < cbase + 64; c0 += 16) {
        uint32_t acc[16];
        tmem_ld16(tmem + lane_off + c0, acc);
        tc_wait_ld();
        float wl[16], ladd[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          wl[i] = inv_den;
          ladd[i] = 0.f;
        }
        if (gl) {  // one branch per trip, not per element
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float w0 = __bfloat162float(gl[(c0 + i) * g_ds]);
            wl[i] = (sig ? __fdividef(1.f, 1.f + __expf(-w0)) : w0) * inv_den;
          }
        }
        if (lnum) {
#pragma unroll
          for (int i = 0; i < 16; ++i) ladd[i] = lnum[c0 + i];
        }
        uint32_t packed[8];
#pragma unroll
        for (int i = 0; i < 16; i += 2)
          packed[i >> 1] = pack_bf16(wl[i] * (__uint_as_float(acc[i]) + ladd[i]),
                                     wl[i + 1] * (__uint_as_float(acc[i + 1]) + ladd[i + 1]));
        // the phi(Q) tile is dead: the output row goes where it was, in the swizzled layout the
        // output tensor map expects
#pragma unroll
        for (int q4 = 0; q4 < 2; ++q4) {
          const int cc = (c0 >> 3) + q4;
          *reinterpret_cast<uint4*>(s_q + (cc >> 3) * kLoHalf + r * 128 + (((cc & 7) ^ (r & 7)) << 4)) =
              make_uint4(packed[4 * q4], packed[4 * q4 + 1], packed[4 * q4 + 2], packed[4 * q4 + 3]);
        }
      }
      if (warp == 2) LO_T(32 + it * 8 + 3);
      tc_fence_before();  // the next tile's MMAs overwrite the accumulator read above
      fence_proxy_async_smem();
      asm volatile("bar.sync 1, %0;" ::"n"(kLoCompute) : "memory");
      if (cw == 0) {
        for (int dh = 0; dh < 2; ++dh) tma_store_3d(&tm_out, s_q + dh * kLoHalf, dh * 64, h, row0);
        tma_store_commit();
        tma_store_wait_read();  // the tile must stay put until it has been read
        LO_T(32 + it * 8 + 4);
        if (it + 1 < my_tiles) load_q(t_begin + it + 1);
      }
    }
    if (cw == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (warp == 2) LO_T(3);
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
  // two CTAs per SM; every CTA of a head walks over the same number of tiles (or one less)
  int splits = (2 * nsm) / p.H;
  if (splits < 1) splits = 1;
  if (splits > n_tiles) splits = n_tiles;
  const int per = (n_tiles + splits - 1) / splits;
  splits = (n_tiles + per - 1) / per;
  dim3 grid(splits, p.H);
  hsa_linear_only_kernel<<<grid, kLoThreads, kLoSmem, st>>>(p, per, tm_q, tm_state, tm_out);
  return cudaGetLastError();
}

}  // namespace hsa
