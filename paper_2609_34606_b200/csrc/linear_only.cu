// Linear branch alone (the "linear only" mode of hsa_forward, head_dim 128):
//   out[i,h] = g_lin * phi(q_i)^T S[h] / (phi(q_i)^T z[h]),   phi(x) = elu(x) + 1
// A lean kernel for the case with no sparse branch: the only traffic is Q in and out out, so it is
// bound by HBM, not by the tensor cores.
// One persistent CTA per SM owns a contiguous run of (head, query tile) items (three at the measured
// size) and asks for the head's state and all of its Q tiles at once, before anything else is set
// up, so that the DRAM latency is paid once.  Roles:
//   warps 0-15  workers, thread = (row, quarter of the dims): phi(q) as packed bf16 into TMEM (the A
//               operand: with A in TMEM the MMAs read only the state from shared memory, which
//               leaves half of its bandwidth to the workers), and later the accumulator ->
//               normalised, gated bf16 row staged where the Q tile was; the loop runs phi(tile i + 1)
//               before the write-out of tile i, so that the tensor cores work on tile i meanwhile
//   warp 16     (one lane) the TMA loads; per tile 32 tcgen05 MMAs phi(Q) S_hi + phi(Q) S_lo and 8 small
//               ones phi(Q) [z_hi z_lo]: the denominator comes out of the tensor cores as two more
//               accumulator columns
//   warp 17     (one lane) TMA store of a finished tile; refills the tile's stage when the run is
//               longer than the ring
// (Q and the output go through shared memory by TMA: per-thread 16-byte global accesses at the
// 3 KB row pitch of a [tokens][H][d] tensor were measured 70 % slower.)
// Every wait is bounded; on expiry the CTA records a timeout and leaves.
#include <cuda_bf16.h>

#include "hsa_internal.h"
#include "ptx.cuh"

namespace hsa {

namespace {

constexpr int kLoStages = 3;                    // Q ring
#ifndef HSA_LO_PARTS
#define HSA_LO_PARTS 2
#endif
constexpr int kLoParts = HSA_LO_PARTS;           // bf16 parts of S fed to the tensor cores: hi + lo
constexpr int kLoSlots = 2;                     // TMEM slots: accumulator + phi(Q) operand
constexpr int kLoWorkers = 512;                 // warps 0..15
constexpr int kLoThreads = kLoWorkers + 64;
constexpr int kLoIssueWarp = kLoWorkers / 32, kLoStoreWarp = kLoIssueWarp + 1;
constexpr int kLoTile = 128 * 128 * 2;          // one [128 x 128] bf16 tile = two swizzled slabs
constexpr int kLoHalf = kLoTile / 2;
constexpr int kLoZop = kZopBytes;               // [16 x 128] bf16 K-major operand: row 0 = z_hi, row 1 = z_lo
constexpr int kLoSmem = (2 + kLoStages) * kLoTile + kLoZop + 512 + 1024;
constexpr uint32_t kLoTmemCols = 512;
constexpr uint32_t kLoSlotCols = 256;           // per slot: 128 numerator columns, 16 for the denominator, 64 of phi(Q)
constexpr uint32_t kLoColDen = 128, kLoColA = 160;

struct LoBars {
  uint64_t q_full[kLoStages];     // Q tile landed
  uint64_t out_ready[kLoStages];  // output tile staged (one arrival per worker warp)
  uint64_t phi_ready[kLoSlots];   // phi(Q) written (one arrival per worker warp)
  uint64_t mma_done[kLoSlots];    // accumulator final, phi(Q) operand dead
  uint64_t acc_free[kLoSlots];    // accumulator read back (one arrival per worker warp)
  uint64_t s_full;                // state tiles and z operand landed
  uint32_t tmem_base;
  volatile int abort_flag;
};
static_assert(sizeof(LoBars) <= 512, "barrier block must fit its shared-memory slot");

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
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(fminf(x * 1.4426950408889634f, 0.f)));
  return fmaxf(x, 0.f) + e;
}

// plain (untiled) bulk copy global -> shared, completion on an mbarrier
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(smem_dst)),
               "l"(reinterpret_cast<uint64_t>(gmem)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

__device__ __forceinline__ void tmem_ld2(uint32_t taddr, uint32_t& r0, uint32_t& r1) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(taddr) : "memory");
}
}  // namespace

// RELU: feature map max(x, 0) instead of elu(x) + 1, and 1e-6 in the denominator (an instance of its
// own: the map sits in the worker warps' innermost loop)
template <bool RELU>
__global__ void __launch_bounds__(kLoThreads, 1)
hsa_linear_only_kernel(FwdParams p, int n_items, const __grid_constant__ CUtensorMap tm_q,
                       const __grid_constant__ CUtensorMap tm_state, const __grid_constant__ CUtensorMap tm_out) {
  constexpr int D = 128;
  extern __shared__ uint8_t lo_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(lo_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* s_state = smem;                        // S_hi | S_lo, MN-major B operands
  uint8_t* s_zop = smem + 2 * kLoTile;            // z operand
  uint8_t* s_ring = smem + 2 * kLoTile + kLoZop;  // Q tile -> output tile, per stage
  LoBars* bars = reinterpret_cast<LoBars*>(smem + (2 + kLoStages) * kLoTile + kLoZop);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tiles = (p.n_q + kTileM - 1) / kTileM;
  // this CTA's run of items (item = head * n_tiles + tile)
  const int i_begin = static_cast<int>(static_cast<int64_t>(blockIdx.x) * n_items / gridDim.x);
  const int i_end = static_cast<int>(static_cast<int64_t>(blockIdx.x + 1) * n_items / gridDim.x);
  const int my_items = i_end - i_begin;

  auto load_q = [&](int it) {
    const int s = it % kLoStages;
    const int item = i_begin + it, h = item / n_tiles, tile = item % n_tiles;
    mbar_expect_tx(&bars->q_full[s], kLoTile);
    for (int dh = 0; dh < 2; ++dh)
      tma_load_3d(s_ring + s * kLoTile + dh * kLoHalf, &tm_q, &bars->q_full[s], dh * 64, h, tile * kTileM);
  };
  auto load_state = [&](int h) {
    mbar_expect_tx(&bars->s_full, kLoParts * kLoTile + kLoZop);
    for (int hl = 0; hl < kLoParts; ++hl) {
      const int rbase = ((h * 2 + p.state_slot) * 2 + hl) * D;
      for (int kb = 0; kb < 2; ++kb)
        for (int dh = 0; dh < 2; ++dh)
          tma_load_2d(s_state + hl * kLoTile + dh * kLoHalf + kb * (kBlock * 128), &tm_state, &bars->s_full, dh * 64,
                      rbase + kb * 64);
    }
    bulk_load(s_zop, p.zop + static_cast<size_t>(h * 2 + p.state_slot) * kLoZop, kLoZop, &bars->s_full);
  };

  // the kernel behind this one may be scheduled as soon as this grid's CTAs have all started
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == kLoIssueWarp * 32) {
    for (int s = 0; s < kLoStages; ++s) {
      mbar_init(&bars->q_full[s], 1);
      mbar_init(&bars->out_ready[s], kLoWorkers / 32);
    }
    for (int a = 0; a < kLoSlots; ++a) {
      mbar_init(&bars->phi_ready[a], kLoWorkers / 32);
      mbar_init(&bars->mma_done[a], 1);
      mbar_init(&bars->acc_free[a], kLoWorkers / 32);
    }
    mbar_init(&bars->s_full, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
    // launched as a programmatic dependent: nothing of the kernel before this one is read earlier
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // every load this CTA will need at first, at once: the DRAM latency is paid once
    if (my_items > 0) {
      load_q(0);
      load_state(i_begin / n_tiles);
      for (int it = 1; it < my_items && it < kLoStages; ++it) load_q(it);
    }
    tma_prefetch_desc(&tm_out);
  }
  if (warp == kLoStoreWarp) {
    tmem_alloc(&bars->tmem_base, kLoTmemCols);
    tmem_relinquish();
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  if (warp == kLoIssueWarp) {
    // ------------------------------------------------------------------ MMA issuer (one lane)
    if (elect_one_sync()) {
      constexpr uint32_t kHiSw = desc_hi_sw128(1024);
      constexpr uint32_t idesc = idesc_bf16_f32(128, D, 0, 1);
      constexpr uint32_t idesc_z = idesc_bf16_f32(128, 16, 0, 0);
      int cur_h = my_items > 0 ? i_begin / n_tiles : -1, s_loads = 0;
      bool s_ok = false;
      for (int it = 0; it < my_items; ++it) {
        const int a = it % kLoSlots;
        const int h = (i_begin + it) / n_tiles;
        if (h != cur_h) {
          // next head: its state replaces the old one once the MMAs that read the old one are done
          if (!lo_wait(&bars->mma_done[(it - 1) % kLoSlots], ((it - 1) / kLoSlots) & 1, bars, p.status)) break;
          load_state(h);
          cur_h = h;
          s_ok = false;
        }
        if (!s_ok) {
          if (!lo_wait(&bars->s_full, s_loads & 1, bars, p.status)) break;
          ++s_loads;
          s_ok = true;
        }
        if (!lo_wait(&bars->phi_ready[a], (it / kLoSlots) & 1, bars, p.status)) break;
        if (it >= kLoSlots && !lo_wait(&bars->acc_free[a], ((it / kLoSlots) - 1) & 1, bars, p.status)) break;
        tc_fence_after();
        const uint32_t acc = tmem + kLoSlotCols * a;
        const uint32_t a_op = acc + kLoColA;  // phi(Q): 16 bf16 of K per 8 columns
        for (int hl = 0; hl < kLoParts; ++hl) {
          const uint32_t b_lo = desc_lo_sw128(smem_u32(s_state + hl * kLoTile), kLoHalf);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk)
            tc_mma_ts_lo(acc, a_op + kk * 8, b_lo + kk * 128, kHiSw, idesc, (hl > 0 || kk > 0) ? 1u : 0u);
        }
        const uint32_t z_lo = desc_lo_sw128(smem_u32(s_zop), 16);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t zoff = ((kk / 4) * (kLoZop / 2) + (kk % 4) * 32) >> 4;
          tc_mma_ts_lo(acc + kLoColDen, a_op + kk * 8, z_lo + zoff, kHiSw, idesc_z, kk > 0 ? 1u : 0u);
        }
        tc_commit(&bars->mma_done[a]);
      }
    }
  } else if (warp == kLoStoreWarp) {
    // ------------------------------------------------------------------ stores + refills (one lane)
    if (elect_one_sync()) {
      for (int it = 0; it < my_items; ++it) {
        const int s = it % kLoStages;
        const int item = i_begin + it, h = item / n_tiles, tile = item % n_tiles;
        if (!lo_wait(&bars->out_ready[s], (it / kLoStages) & 1, bars, p.status)) break;
        uint8_t* s_q = s_ring + s * kLoTile;
        for (int dh = 0; dh < 2; ++dh) tma_store_3d(&tm_out, s_q + dh * kLoHalf, dh * 64, h, tile * kTileM);
        tma_store_commit();
        if (it + kLoStages < my_items) {
          tma_store_wait_read();  // the tile must stay put until it has been read
          load_q(it + kLoStages);
        }
      }
      tma_store_wait_read();  // shared memory may go once the stores have read it
    }
  } else {
    // ------------------------------------------------------------------ workers
    // thread = (row, quarter of the dims): the same cells of the stage hold its Q and its output;
    // the row is also its TMEM lane
    const int quad = warp & 3, cq = warp >> 2;
    const int r = quad * 32 + lane;
    const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
    uint32_t cell[4];  // byte offsets of the thread's four 16-byte chunks inside a stage
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int cc = cq * 4 + i;
      cell[i] = (cc >> 3) * kLoHalf + r * 128 + (((cc & 7) ^ (r & 7)) << 4);
    }
    const bool sig = p.gate_act == 1;
    const bool plain = p.g_lin == nullptr && p.lin_num == nullptr;  // no gate, no causal partials
    bool ok = true;
#pragma unroll 1
    for (int it = 0; it <= my_items && ok; ++it) {
      if (it < my_items) {
        // ---- phi of tile it into TMEM slot it % 2 (its last reader, the MMAs of tile it - 2, is done:
        // the write-out of that tile, which waited for them, comes earlier in this loop)
        const int s = it % kLoStages;
        ok = lo_wait(&bars->q_full[s], (it / kLoStages) & 1, bars, p.status);
        if (!ok) break;
        const uint8_t* s_q = s_ring + s * kLoTile;
        uint4 raw[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) raw[i] = *reinterpret_cast<const uint4*>(s_q + cell[i]);
        uint32_t o[16];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t* qw = reinterpret_cast<const uint32_t*>(&raw[i]);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float x0 = __uint_as_float(qw[e] << 16), x1 = __uint_as_float(qw[e] & 0xffff0000u);
            o[4 * i + e] = RELU ? pack_bf16(fmaxf(x0, 0.f), fmaxf(x1, 0.f)) : pack_bf16(lo_phi(x0), lo_phi(x1));
          }
        }
        // this thread's 32 values of phi(q) are 16 columns of its TMEM lane
        tmem_st16(tmem + lane_off + kLoSlotCols * (it % kLoSlots) + kLoColA + cq * 16, o);
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->phi_ready[it % kLoSlots]);
      }
      if (it >= 1) {
        // ---- write-out of tile it - 1
        const int jt = it - 1;
        const int s = jt % kLoStages, a = jt % kLoSlots;
        const int item = i_begin + jt, h = item / n_tiles, tile = item % n_tiles;
        const int row = tile * kTileM + r;
        uint8_t* s_q = s_ring + s * kLoTile;
        ok = lo_wait(&bars->mma_done[a], (jt / kLoSlots) & 1, bars, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t acc = tmem + lane_off + kLoSlotCols * a;
        uint32_t v[32], d0, d1;
        tmem_ld32(acc + cq * 32, v);
        tmem_ld2(acc + kLoColDen, d0, d1);
        tc_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->acc_free[a]);
        float den = __uint_as_float(d0) + __uint_as_float(d1);
        const bool wr = row < p.n_q;  // rows past the end of the chunk compute but never store
        uint32_t packed[16];
        if (plain) {
          const float inv_den = RELU ? 1.f / (den + 1e-6f) : (den > 0.f ? 1.f / den : 0.f);
#pragma unroll
          for (int i = 0; i < 32; i += 2)
            packed[i >> 1] = pack_bf16(__uint_as_float(v[i]) * inv_den, __uint_as_float(v[i + 1]) * inv_den);
        } else {
          const float* lnum = nullptr;
          if (wr && p.lin_num != nullptr) {
            lnum = p.lin_num + (static_cast<size_t>(row) * p.H + h) * D + cq * 32;
            den += p.lin_den[static_cast<size_t>(row) * p.H + h];
          }
          const float inv_den = RELU ? 1.f / (den + 1e-6f) : (den > 0.f ? 1.f / den : 0.f);
          const __nv_bfloat16* gl =
              (wr && p.g_lin) ? p.g_lin + static_cast<size_t>(row) * p.g_ts + static_cast<size_t>(h) * p.g_hs : nullptr;
          const int g_ds = static_cast<int>(p.g_ds);
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            float w0 = inv_den, w1 = inv_den, l0 = 0.f, l1 = 0.f;
            if (gl) {
              const float g0 = __bfloat162float(gl[(cq * 32 + i) * g_ds]), g1 = __bfloat162float(gl[(cq * 32 + i + 1) * g_ds]);
              w0 *= sig ? __fdividef(1.f, 1.f + __expf(-g0)) : g0;
              w1 *= sig ? __fdividef(1.f, 1.f + __expf(-g1)) : g1;
            }
            if (lnum) {
              l0 = lnum[i];
              l1 = lnum[i + 1];
            }
            packed[i >> 1] = pack_bf16(w0 * (__uint_as_float(v[i]) + l0), w1 * (__uint_as_float(v[i + 1]) + l1));
          }
        }
        // the Q tile is dead (each thread has read its own cells): the output row goes where it was,
        // in the swizzled layout the output tensor map expects
#pragma unroll
        for (int i = 0; i < 4; ++i)
          *reinterpret_cast<uint4*>(s_q + cell[i]) =
              make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->out_ready[s]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kLoStoreWarp) {
    tc_fence_after();
    tmem_dealloc(tmem, kLoTmemCols);
  }
}

cudaError_t linear_only_init() {
  cudaError_t e = cudaFuncSetAttribute(hsa_linear_only_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kLoSmem);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(hsa_linear_only_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kLoSmem);
  return e;
}

cudaError_t launch_linear_only(const FwdParams& p, int nsm, const CUtensorMap& tm_q, const CUtensorMap& tm_state,
                               const CUtensorMap& tm_out, cudaStream_t st) {
  const int n_tiles = (p.n_q + kTileM - 1) / kTileM;
  const int n_items = n_tiles * p.H;
  const int grid = n_items < nsm ? n_items : nsm;  // one persistent CTA per SM
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kLoThreads);
  cfg.dynamicSmemBytes = kLoSmem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (p.relu) return cudaLaunchKernelEx(&cfg, hsa_linear_only_kernel<true>, p, n_items, tm_q, tm_state, tm_out);
  return cudaLaunchKernelEx(&cfg, hsa_linear_only_kernel<false>, p, n_items, tm_q, tm_state, tm_out);
}

}  // namespace hsa
