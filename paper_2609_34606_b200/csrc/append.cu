// hsa_append_kv kernels: pool write + per-block key sums, and the linear-branch state update
//   S[h] += sum_j phi(k_j)^T v_j,   z[h] += sum_j phi(k_j),   phi(x) = elu(x) + 1
// as a deterministic two-stage reduction (no floating-point atomics).
#include <cuda_bf16.h>

#include "hsa_internal.h"
#include "ptx.cuh"

namespace hsa {

__device__ __forceinline__ float phi_elu1(float x) { return x > 0.f ? x + 1.f : expf(x); }

// ---------------------------------------------------------------------------------------
// Stage A: one CTA per (touched block, head).  Copies the new rows of K and V into the block's
// page and adds their column sums to the block's key sum.  A CTA owns its (head, block)
// exclusively, so the sum order is fixed.
// ---------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) append_pool_ksum_kernel(AppendArgs a) {
  constexpr int CH = D / 8;     // 16-byte chunks per row
  constexpr int RP = 256 / CH;  // rows handled per pass
  __shared__ float red[RP][D];

  const int h = blockIdx.y;
  const int64_t b = a.n0 / kBlock + blockIdx.x;
  const int64_t t_lo = max(a.n0, b * kBlock);
  const int64_t t_hi = min(a.n0 + a.n_new, b * kBlock + kBlock);
  const int c8 = threadIdx.x % CH;
  const int rg = threadIdx.x / CH;
  const int page = a.page_table[b];
  const size_t row_base = (static_cast<size_t>(page) * a.H + h) * kBlock;

  float acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.f;

  for (int64_t t = t_lo + rg; t < t_hi; t += RP) {
    const size_t src = static_cast<size_t>(t - a.n0) * a.tok_stride +
                       static_cast<size_t>(h) * a.head_stride + c8 * 8;
    const uint4 kk = *reinterpret_cast<const uint4*>(a.k + src);
    const uint4 vv = *reinterpret_cast<const uint4*>(a.v + src);
    const size_t dst = (row_base + (t - b * kBlock)) * D + c8 * 8;
    *reinterpret_cast<uint4*>(a.k_pool + dst) = kk;
    *reinterpret_cast<uint4*>(a.v_pool + dst) = vv;
    const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&kk);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(k2[i]);
      acc[2 * i] += f.x;
      acc[2 * i + 1] += f.y;
    }
  }
  // Rows of a partial tail page past the last token are zero-filled: the forward kernel masks
  // their scores, but 0 * (uninitialised V) must not be able to produce a NaN.
  for (int64_t t = t_hi + rg; t < b * kBlock + kBlock; t += RP) {
    const size_t dst = (row_base + (t - b * kBlock)) * D + c8 * 8;
    *reinterpret_cast<uint4*>(a.k_pool + dst) = make_uint4(0, 0, 0, 0);
    *reinterpret_cast<uint4*>(a.v_pool + dst) = make_uint4(0, 0, 0, 0);
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) red[rg][c8 * 8 + i] = acc[i];
  __syncthreads();
  if (threadIdx.x < D) {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < RP; ++r) s += red[r][threadIdx.x];
    float* dst = a.ksum + (static_cast<size_t>(h) * a.max_pages + b) * D + threadIdx.x;
    float old = 0.f;
    if (t_lo > b * kBlock) {  // block already partly filled: its sum before this append
      float* saved = a.ksum_saved + static_cast<size_t>(h) * D + threadIdx.x;
      old = a.tail_from_saved ? *saved : *dst;
      if (!a.tail_from_saved) *saved = old;
    }
    *dst = old + s;
  }
  // Launched as a programmatic dependent (Linformer form: behind the compression kernel, whose
  // outputs it does not touch) this grid runs beside that kernel and waits for it only here, so
  // that its own end implies that kernel's.  Launched normally this is a no-op.
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ---------------------------------------------------------------------------------------
// Stage B: partial state over a token range.  grid (nsplit, H), 256 threads; each thread owns a
// register tile of the D x D outer-product sum.
// ---------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) state_partial_kernel(AppendArgs a) {
  constexpr int TB = 32;       // tokens staged per batch
  constexpr int R = D / 32;    // 4 (D=128) or 2 (D=64): half-tile edge
  __shared__ __align__(16) float fk[TB][D];
  __shared__ __align__(16) float vv[TB][D];

  const int h = blockIdx.y;
  const int split = blockIdx.x;
  const int per = (a.n_new + a.nsplit - 1) / a.nsplit;
  const int t0 = split * per;
  const int t1 = min(a.n_new, t0 + per);
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  // thread tile: rows {ty*R + i, D/2 + ty*R + i}, cols {tx*R + j, D/2 + tx*R + j}
  float acc[2 * R][2 * R];
#pragma unroll
  for (int i = 0; i < 2 * R; ++i)
#pragma unroll
    for (int j = 0; j < 2 * R; ++j) acc[i][j] = 0.f;
  float zacc = 0.f;

  constexpr int CH = D / 8;
  for (int tb = t0; tb < t1; tb += TB) {
    const int nt = min(TB, t1 - tb);
    __syncthreads();
    for (int idx = threadIdx.x; idx < TB * CH; idx += 256) {
      const int r = idx / CH, c8 = idx % CH;
      float kf[8], vf[8];
      if (r < nt) {
        const size_t src = static_cast<size_t>(tb + r) * a.tok_stride +
                           static_cast<size_t>(h) * a.head_stride + c8 * 8;
        const uint4 kk = *reinterpret_cast<const uint4*>(a.k + src);
        const uint4 v4 = *reinterpret_cast<const uint4*>(a.v + src);
        const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&kk);
        const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&v4);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __bfloat1622float2(k2[i]);
          const float2 g = __bfloat1622float2(v2[i]);
          kf[2 * i] = a.relu ? fmaxf(f.x, 0.f) : phi_elu1(f.x);
          kf[2 * i + 1] = a.relu ? fmaxf(f.y, 0.f) : phi_elu1(f.y);
          vf[2 * i] = g.x;
          vf[2 * i + 1] = g.y;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) kf[i] = vf[i] = 0.f;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        fk[r][c8 * 8 + i] = kf[i];
        vv[r][c8 * 8 + i] = vf[i];
      }
    }
    __syncthreads();
    if (threadIdx.x < D) {
#pragma unroll 8
      for (int r = 0; r < TB; ++r) zacc += fk[r][threadIdx.x];
    }
#pragma unroll 4
    for (int r = 0; r < TB; ++r) {
      float ka[2 * R], va[2 * R];
#pragma unroll
      for (int i = 0; i < R; ++i) {
        ka[i] = fk[r][ty * R + i];
        ka[R + i] = fk[r][D / 2 + ty * R + i];
        va[i] = vv[r][tx * R + i];
        va[R + i] = vv[r][D / 2 + tx * R + i];
      }
#pragma unroll
      for (int i = 0; i < 2 * R; ++i)
#pragma unroll
        for (int j = 0; j < 2 * R; ++j) acc[i][j] = fmaf(ka[i], va[j], acc[i][j]);
    }
  }
  float* out = a.spart + (static_cast<size_t>(h) * a.nsplit + split) * (D * D + D);
#pragma unroll
  for (int i = 0; i < 2 * R; ++i) {
    const int row = (i < R) ? ty * R + i : D / 2 + ty * R + (i - R);
#pragma unroll
    for (int j = 0; j < 2 * R; ++j) {
      const int col = (j < R) ? tx * R + j : D / 2 + tx * R + (j - R);
      out[row * D + col] = acc[i][j];
    }
  }
  if (threadIdx.x < D) out[D * D + threadIdx.x] = zacc;
}

// ---------------------------------------------------------------------------------------
// Stage C: S[dst] <- S[src] + sum of partials (fixed order), with its bf16 hi/lo split (the forward
// kernels feed hi and lo to the tensor cores as two bf16 operands), the same for z and its operand image.
// ---------------------------------------------------------------------------------------
__global__ void state_reduce_kernel(AppendArgs a) {
  const int D = a.D;
  const int DD = D * D;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  const int h = blockIdx.y;
  if (idx >= DD + D) return;
  // results of the kernel before this one are needed from here on
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const float* part = a.spart + static_cast<size_t>(h) * a.nsplit * (DD + D) + idx;
  // all partials are fetched at once (independent loads in flight); the sum order stays fixed
  float v[kStateSplitMax];
#pragma unroll
  for (int i = 0; i < kStateSplitMax; ++i)
    v[i] = (i < a.nsplit) ? __ldcg(&part[static_cast<size_t>(i) * (DD + D)]) : 0.f;
  float add = 0.f;
#pragma unroll
  for (int i = 0; i < kStateSplitMax; ++i) add += v[i];
  const int dst = a.src_slot ^ 1;
  if (idx < DD) {
    const size_t o = static_cast<size_t>(h) * DD + idx;
    const float s_new = a.S[a.src_slot][o] + add;
    a.S[dst][o] = s_new;
    __nv_bfloat16* hl = a.hilo + (static_cast<size_t>(h) * 2 + dst) * 2 * DD + idx;
    const __nv_bfloat16 nh = __float2bfloat16_rn(s_new);
    hl[0] = nh;
    hl[DD] = __float2bfloat16_rn(s_new - __bfloat162float(nh));
  } else {
    const int k = idx - DD;
    const size_t o = static_cast<size_t>(h) * D + k;
    const float z_new = a.z[a.src_slot][o] + add;
    a.z[dst][o] = z_new;
    if (D == 128) {
      // operand image of z: element (row n, dim k) of a K-major tile with the 128-byte swizzle sits
      // at slab (k / 64), row n, 16-byte chunk ((k % 64) / 8) ^ (n % 8)
      const int slab = k >> 6, kk = k & 63, c = kk >> 3;
      uint8_t* img = a.zop + static_cast<size_t>(h * 2 + dst) * kZopBytes + slab * (kZopBytes / 2) + (kk & 7) * 2;
      const __nv_bfloat16 hi = __float2bfloat16_rn(z_new);
      *reinterpret_cast<__nv_bfloat16*>(img + 0 * 128 + ((c ^ 0) << 4)) = hi;
      *reinterpret_cast<__nv_bfloat16*>(img + 1 * 128 + ((c ^ 1) << 4)) = __float2bfloat16_rn(z_new - __bfloat162float(hi));
    }
  }
}

// ---------------------------------------------------------------------------------------
// Fused append for head_dim 128 (the measured path): one pass over the chunk's K and V in which
// no thread touches global memory for the bulk data.
// grid (nsplit, H); a CTA owns a run of consecutive history blocks of one head.  Per block
//   * the producer lane brings the block's rows of K and V into a 4-deep ring by TMA (rows
//     outside the chunk arrive as zeros) and sends the same tiles on to the block's page by
//     TMA store (a block that already held tokens before this call is written row by row by
//     the workers instead, so that its old rows stay),
//   * sixteen worker warps (two groups on alternate blocks) read K from the ring, build phi(K) as bf16 hi + lo (hi + lo carries
//     ~16 bits) in the 128-byte-swizzled MN-major layout,
//   * the MMA lane lets the tensor cores accumulate, over the block's tokens (tcgen05, K = tokens)
//       S_part (128 x 128, fp32 in TMEM) += phi(K)_hi^T V + phi(K)_lo^T V      (V straight from the ring)
//       z_part (128 x 16)                 += phi(K)_hi^T 1 + phi(K)_lo^T 1
//       ksum_b (128 x 16)                  = K^T 1                              (K straight from the ring)
//     and four more warps read ksum_b back as soon as it is final,
// and finally the CTA writes its partial S and z for the fixed-order reduction of stage C.
// Every wait is bounded; on expiry the CTA records a timeout and leaves.
// ---------------------------------------------------------------------------------------

namespace {

constexpr int kAfDepth = 4;                      // ring stages
constexpr int kAfWorkers = 512;                  // worker threads (warps 2..17)
constexpr int kAfThreads = 64 + kAfWorkers + 128;  // + producer warp + MMA warp + 4 key-sum warps
constexpr int kAfTile = 64 * 128 * 2;            // [64 tokens x 128 dims] bf16 = two swizzled slabs
constexpr int kAfStage = 2 * kAfTile;            // K | V
constexpr int kAfHilo = 2 * kAfTile;             // phi hi | phi lo
constexpr int kAfOnes = 2048;                    // [16 x 64] bf16 ones (K-major operand)
constexpr int kAfSmem = kAfDepth * kAfStage + 2 * kAfHilo + kAfOnes + 256 + 1024;
constexpr uint32_t kAfTmemCols = 256;
constexpr uint32_t kAfColZ = 128, kAfColKs = 144;  // TMEM columns: S 0..127, z, ksum[2]
constexpr int kAfPitch = 132;                      // floats per row of the staged partial state
static_assert(128 * kAfPitch * 4 <= 2 * kAfHilo + kAfOnes, "partial state is staged in the hi/lo + ones area");

struct AfBars {
  uint64_t full[kAfDepth];      // ring stage landed
  uint64_t consumed[kAfDepth];  // tensor cores are done with the stage
  uint64_t phi_ready[2];        // hi/lo buffer written
  uint64_t mma_done[2];         // tensor cores are done with the hi/lo buffer (and ksum is final)
  uint64_t ks_read[2];          // key-sum buffer read back
  uint32_t tmem_base;
  volatile int abort_flag;
};

__device__ __forceinline__ bool af_wait(uint64_t* bar, uint32_t parity, AfBars* bars, int32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  for (uint32_t i = 1; i < (1u << 24); ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 0u && bars->abort_flag) return false;
  }
  bars->abort_flag = 1;
  atomicCAS(status, 0, kDevTimeout);
  return false;
}

// elu(x) + 1 with the fast exponential (relative error ~1e-6, far inside the state's tolerance)
__device__ __forceinline__ float phi_fast(float x) {
  float e;  // branch-free: elu(x) + 1 = max(x, 0) + exp(min(x, 0))
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(fminf(x, 0.f) * 1.4426950408889634f));
  return fmaxf(x, 0.f) + e;
}

__device__ __forceinline__ void tma_store_2d(const void* tmap, const void* smem_src, int32_t x, int32_t y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                   reinterpret_cast<uint64_t>(tmap)),
               "r"(smem_u32(smem_src)), "r"(x), "r"(y)
               : "memory");
}

}  // namespace

// RELU: the feature map is max(x, 0) instead of elu(x) + 1 (an instance of its own: the map sits in
// the innermost loop of the worker warps)
template <bool RELU>
__global__ void __launch_bounds__(kAfThreads, 1)
append_fused_kernel(AppendArgs a, int blocks_per_cta, const __grid_constant__ CUtensorMap tm_kin,
                    const __grid_constant__ CUtensorMap tm_vin, const __grid_constant__ CUtensorMap tm_kpool,
                    const __grid_constant__ CUtensorMap tm_vpool) {
  constexpr int D = 128;
  extern __shared__ uint8_t af_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(af_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* ring = smem;
  uint8_t* hilo = smem + kAfDepth * kAfStage;
  uint8_t* ones = hilo + 2 * kAfHilo;
  AfBars* bars = reinterpret_cast<AfBars*>(ones + kAfOnes);

  // the reduction kernel behind this one may be scheduled early; it waits for this grid itself
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // This grid is itself launched as a programmatic dependent: it may be scheduled while the kernel
  // before it in the stream (the forward kernel of the layer before) is still finishing.  The
  // set-up below touches nothing of that kernel's; every thread waits for its end (wait_prior)
  // before the first load of the inputs is issued and before the CTA-wide barrier.
  auto wait_prior = [] { asm volatile("griddepcontrol.wait;" ::: "memory"); };

  const int h = blockIdx.y, split = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t b_first = a.n0 / kBlock, b_last = (a.n0 + a.n_new - 1) / kBlock;
  const int64_t bs = b_first + static_cast<int64_t>(split) * blocks_per_cta;
  const int64_t be = min64(b_last + 1, bs + blocks_per_cta);
  const int nblk = static_cast<int>(max64(0, be - bs));
  const int64_t n_end = a.n0 + a.n_new;

  auto issue_loads = [&](int bi) {
    const int s = bi % kAfDepth;
    uint8_t* st = ring + s * kAfStage;
    const int32_t row0 = static_cast<int32_t>((bs + bi) * kBlock - a.n0);  // may be negative: zero fill
    mbar_expect_tx(&bars->full[s], kAfStage);
    tma_load_3d(st, &tm_kin, &bars->full[s], 0, h, row0);
    tma_load_3d(st + kAfTile / 2, &tm_kin, &bars->full[s], 64, h, row0);
    tma_load_3d(st + kAfTile, &tm_vin, &bars->full[s], 0, h, row0);
    tma_load_3d(st + kAfTile + kAfTile / 2, &tm_vin, &bars->full[s], 64, h, row0);
  };
  if (threadIdx.x == 0) {
    for (int s = 0; s < kAfDepth; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->consumed[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->phi_ready[s], kAfWorkers / 2);  // one worker group per buffer
      mbar_init(&bars->mma_done[s], 1);
      mbar_init(&bars->ks_read[s], 4);
    }
    bars->abort_flag = 0;
    fence_mbar_init();
    wait_prior();
    // the first ring fill starts before the rest of the CTA is set up
    for (int bi = 0; bi < nblk && bi < kAfDepth; ++bi) issue_loads(bi);
    tma_prefetch_desc(&tm_kpool);
    tma_prefetch_desc(&tm_vpool);
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, kAfTmemCols);
    tmem_relinquish();
  }
  // bf16 1.0 everywhere: under any swizzle the tile reads as all ones
  for (int i = threadIdx.x; i < kAfOnes / 4; i += kAfThreads) reinterpret_cast<uint32_t*>(ones)[i] = 0x3F803F80u;
  fence_proxy_async_smem();
  wait_prior();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer (one lane)
    if (elect_one_sync()) {
      bool ok = true;
      for (int bi = 0; bi < nblk && ok; ++bi) {
        const int s = bi % kAfDepth;
        ok = af_wait(&bars->full[s], (bi / kAfDepth) & 1, bars, a.status);
        if (!ok) break;
        const int64_t b = bs + bi;
        if (b * kBlock >= a.n0) {  // the block holds nothing older: whole tiles go to its page
          uint8_t* st = ring + s * kAfStage;
          const int32_t prow = (a.page_table[b] * a.H + h) * kBlock;
          tma_store_2d(&tm_kpool, st, 0, prow);
          tma_store_2d(&tm_kpool, st + kAfTile / 2, 64, prow);
          tma_store_2d(&tm_vpool, st + kAfTile, 0, prow);
          tma_store_2d(&tm_vpool, st + kAfTile + kAfTile / 2, 64, prow);
        }
        tma_store_commit();
        if (bi >= 1 && bi - 1 + kAfDepth < nblk) {
          // refill the stage of block bi - 1: its stores have read it, the tensor cores are done
          asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
          ok = af_wait(&bars->consumed[(bi - 1) % kAfDepth], ((bi - 1) / kAfDepth) & 1, bars, a.status);
          if (ok) issue_loads(bi - 1 + kAfDepth);
        }
      }
      asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // every page write has landed
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (one lane)
    if (elect_one_sync()) {
      constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 1, 1);
      constexpr uint32_t idesc_1 = idesc_bf16_f32(128, 16, 1, 0);
      constexpr uint32_t hi = desc_hi_sw128(1024);
      const uint32_t b_ones = desc_lo_sw128(smem_u32(ones), 16);
      for (int bi = 0; bi < nblk; ++bi) {
        const int s = bi % kAfDepth, hb = bi & 1;
        if (!af_wait(&bars->phi_ready[hb], (bi >> 1) & 1, bars, a.status)) break;
        tc_fence_after();
        uint8_t* st = ring + s * kAfStage;
        const uint32_t a_k = desc_lo_sw128(smem_u32(st), kAfTile / 2);
        const uint32_t b_v = desc_lo_sw128(smem_u32(st + kAfTile), kAfTile / 2);
        const uint32_t a_hi = desc_lo_sw128(smem_u32(hilo + hb * kAfHilo), kAfTile / 2);
        const uint32_t a_lo = desc_lo_sw128(smem_u32(hilo + hb * kAfHilo + kAfTile), kAfTile / 2);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_ss_lo(tmem, a_hi + kk * 128, b_v + kk * 128, hi, idesc_s, (bi > 0 || kk > 0) ? 1u : 0u);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) tc_mma_ss_lo(tmem, a_lo + kk * 128, b_v + kk * 128, hi, idesc_s, 1u);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_ss_lo(tmem + kAfColZ, a_hi + kk * 128, b_ones, hi, idesc_1, (bi > 0 || kk > 0) ? 1u : 0u);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) tc_mma_ss_lo(tmem + kAfColZ, a_lo + kk * 128, b_ones, hi, idesc_1, 1u);
        if (bi >= 2 && !af_wait(&bars->ks_read[hb], ((bi >> 1) - 1) & 1, bars, a.status)) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_ss_lo(tmem + kAfColKs + hb * 16, a_k + kk * 128, b_ones, hi, idesc_1, kk > 0 ? 1u : 0u);
        tc_commit(&bars->consumed[s]);
        tc_commit(&bars->mma_done[hb]);
      }
    }
  } else if (warp >= 2 + kAfWorkers / 32) {
    // ------------------------------------------------------------------ key-sum warps
    // one warp per TMEM lane quadrant: key sum of each block, as soon as its MMAs are done
    const int quad = warp & 3;
    for (int bj = 0; bj < nblk; ++bj) {
      if (!af_wait(&bars->mma_done[bj & 1], (bj >> 1) & 1, bars, a.status)) break;
      tc_fence_after();
      uint32_t v[16];
      tmem_ld16(tmem + (static_cast<uint32_t>(quad * 32) << 16) + kAfColKs + (bj & 1) * 16, v);
      tc_wait_ld();
      tc_fence_before();
      if (lane == 0) mbar_arrive(&bars->ks_read[bj & 1]);
      const int64_t b = bs + bj;
      float* dst = a.ksum + (static_cast<size_t>(h) * a.max_pages + b) * D + quad * 32 + lane;
      float old = 0.f;
      if (a.n0 > b * kBlock) {  // block partly filled before: its sum before this append
        float* saved = a.ksum_saved + static_cast<size_t>(h) * D + quad * 32 + lane;
        old = a.tail_from_saved ? *saved : *dst;
        if (!a.tail_from_saved) *saved = old;
      }
      *dst = old + __uint_as_float(v[0]);
    }
  } else {
    // ------------------------------------------------------------------ workers
    // two groups of eight warps take alternate blocks, so that one group's waits hide under the
    // other's arithmetic
    const int w = threadIdx.x - 64;
    const int grp = w >> 8, wg = w & 255;
    const int ch = wg & 15;  // 16-byte chunk of a row (8 dims)
    const int rg = wg >> 4;  // rows rg, rg + 16, rg + 32, rg + 48 of a block
    const int quad = warp & 3;
    bool ok = true;
    uint32_t soff[4];  // the thread's four 16-byte chunks inside a swizzled [64 x 128] tile
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = rg + 16 * i;
      soff[i] = (ch >> 3) * (kAfTile / 2) + r * 128 + (((ch & 7) ^ (r & 7)) << 4);
    }
#pragma unroll 1
    for (int bi = grp; bi < nblk && ok; bi += 2) {
      const int s = bi % kAfDepth, hb = bi & 1;
      const int64_t b = bs + bi;
      ok = af_wait(&bars->full[s], (bi / kAfDepth) & 1, bars, a.status);
      if (!ok) break;
      const uint8_t* st_k = ring + s * kAfStage;
      uint4 kreg[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) kreg[i] = *reinterpret_cast<const uint4*>(st_k + soff[i]);
      if (b * kBlock < a.n0) {
        // block partly filled before this call: only its new rows (and the zero rows past the
        // last token) are written, by hand
        const size_t row_base = (static_cast<size_t>(a.page_table[b]) * a.H + h) * kBlock;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int r = rg + 16 * i;
          const int64_t t = b * kBlock + r;
          if (t >= a.n0) {
            const size_t dst = (row_base + r) * D + ch * 8;
            *reinterpret_cast<uint4*>(a.k_pool + dst) = kreg[i];
            *reinterpret_cast<uint4*>(a.v_pool + dst) = *reinterpret_cast<const uint4*>(st_k + kAfTile + soff[i]);
          }
        }
      }
      if (bi >= 2) {
        ok = af_wait(&bars->mma_done[hb], ((bi >> 1) - 1) & 1, bars, a.status);
        if (!ok) break;
      }
      uint8_t* st_hi = hilo + hb * kAfHilo;
      uint8_t* st_lo = st_hi + kAfTile;
      // rows outside the chunk (only in its first and last block) add nothing to the state
      const bool whole = b * kBlock >= a.n0 && b * kBlock + kBlock <= n_end;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t* kw = reinterpret_cast<const uint32_t*>(&kreg[i]);
        uint32_t hw[4], lw[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float x0 = __uint_as_float(kw[e] << 16), x1 = __uint_as_float(kw[e] & 0xffff0000u);
          const float p0 = RELU ? fmaxf(x0, 0.f) : phi_fast(x0);
          const float p1 = RELU ? fmaxf(x1, 0.f) : phi_fast(x1);
          hw[e] = pack_bf16(p0, p1);
          lw[e] = pack_bf16(p0 - __uint_as_float(hw[e] << 16), p1 - __uint_as_float(hw[e] & 0xffff0000u));
        }
        if (!whole) {
          const int64_t t = b * kBlock + rg + 16 * i;
          if (t < a.n0 || t >= n_end) {
#pragma unroll
            for (int e = 0; e < 4; ++e) hw[e] = lw[e] = 0u;
          }
        }
        *reinterpret_cast<uint4*>(st_hi + soff[i]) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
        *reinterpret_cast<uint4*>(st_lo + soff[i]) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
      }
      fence_proxy_async_smem();  // generic-proxy writes above -> visible to the tensor cores
      mbar_arrive(&bars->phi_ready[hb]);
    }
    // the partial state, once every MMA is done: the last two blocks' barriers, in block order (a
    // group has not watched the other group's barrier, so it must not skip a phase of it)
    for (int bj = max(0, nblk - 2); bj < nblk && ok; ++bj)
      ok = af_wait(&bars->mma_done[bj & 1], (bj >> 1) & 1, bars, a.status);
    tc_fence_after();
    float* out = a.spart + (static_cast<size_t>(h) * a.nsplit + split) * (D * D + D);
    const int row = quad * 32 + lane;
    {
      // TMEM -> shared memory (row pitch 132 floats: conflict-free both ways) -> coalesced rows
      float* stage = reinterpret_cast<float*>(hilo);
      uint32_t v[32];
      const int col = ((warp - 2) >> 2) * 32;  // four warps per lane quadrant, 32 columns each
      if (nblk > 0 && ok) {
        tmem_ld32(tmem + (static_cast<uint32_t>(quad * 32) << 16) + col, v);
        tc_wait_ld();
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = 0u;
      }
      float4* srow = reinterpret_cast<float4*>(stage + row * kAfPitch + col);
#pragma unroll
      for (int i = 0; i < 8; ++i)
        srow[i] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                              __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
      asm volatile("bar.sync 1, %0;" ::"n"(kAfWorkers) : "memory");
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int f = w + kAfWorkers * i;  // float4 index of the [128][128] partial state
        const int r2 = f >> 5, c4 = f & 31;
        reinterpret_cast<float4*>(out)[f] = *reinterpret_cast<const float4*>(stage + r2 * kAfPitch + c4 * 4);
      }
    }
    if (warp < 6) {
      uint32_t v[16];
      v[0] = 0u;
      if (nblk > 0 && ok) {
        tmem_ld16(tmem + (static_cast<uint32_t>(quad * 32) << 16) + kAfColZ, v);
        tc_wait_ld();
      }
      out[D * D + row] = __uint_as_float(v[0]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kAfTmemCols);
  }
}

cudaError_t append_init() {
  cudaError_t e = cudaFuncSetAttribute(append_fused_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAfSmem);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(append_fused_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAfSmem);
  return e;
}

cudaError_t launch_append(const AppendArgs& a_in, const AppendMaps* maps, cudaStream_t st) {
  AppendArgs a = a_in;
  const int64_t b0 = a.n0 / kBlock;
  const int64_t b1 = (a.n0 + a.n_new - 1) / kBlock;
  cudaError_t e;
  if (a.D == 128 && a.lin_state && maps) {
    const int nb = static_cast<int>(b1 - b0 + 1);
    const int per = (nb + a.nsplit - 1) / a.nsplit;
    a.nsplit = (nb + per - 1) / per;  // no empty CTAs
    dim3 grid(a.nsplit, a.H);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kAfThreads);
    cfg.dynamicSmemBytes = kAfSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (a.relu)
      e = cudaLaunchKernelEx(&cfg, append_fused_kernel<true>, a, per, maps->kin, maps->vin, maps->kpool, maps->vpool);
    else
      e = cudaLaunchKernelEx(&cfg, append_fused_kernel<false>, a, per, maps->kin, maps->vin, maps->kpool, maps->vpool);
    if (e != cudaSuccess) return e;
  } else {
    dim3 gridA(static_cast<unsigned>(b1 - b0 + 1), a.H);
    cudaLaunchConfig_t cfgA{};
    cfgA.gridDim = gridA;
    cfgA.blockDim = dim3(256);
    cfgA.stream = st;
    cudaLaunchAttribute attrA[1];
    attrA[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrA[0].val.programmaticStreamSerializationAllowed = 1;
    cfgA.attrs = attrA;
    cfgA.numAttrs = a.beside_prior ? 1 : 0;  // (only behind a kernel whose outputs this one leaves alone)
    if (a.D == 128)
      e = cudaLaunchKernelEx(&cfgA, append_pool_ksum_kernel<128>, a);
    else
      e = cudaLaunchKernelEx(&cfgA, append_pool_ksum_kernel<64>, a);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess || !a.lin_state) return e;
    dim3 gridB(a.nsplit, a.H);
    if (a.D == 128)
      state_partial_kernel<128><<<gridB, 256, 0, st>>>(a);
    else
      state_partial_kernel<64><<<gridB, 256, 0, st>>>(a);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  // The reduction may be scheduled while the kernel before it drains (programmatic dependent
  // launch); it waits for that kernel's results itself before it reads anything.
  const int n = a.D * a.D + a.D;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((n + 255) / 256, a.H);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, state_reduce_kernel, a);
}

}  // namespace hsa
