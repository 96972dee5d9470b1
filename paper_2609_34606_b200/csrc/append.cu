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
    const float old = (t_lo > b * kBlock) ? *dst : 0.f;  // block already partly filled
    *dst = old + s;
  }
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
          kf[2 * i] = phi_elu1(f.x);
          kf[2 * i + 1] = phi_elu1(f.y);
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
// Stage C: S_prev <- S, S <- S + sum of partials (fixed order), and the bf16 hi/lo split of
// both (the forward kernel feeds hi and lo to the tensor cores as two bf16 operands).
// ---------------------------------------------------------------------------------------
__global__ void state_reduce_kernel(AppendArgs a) {
  const int D = a.D;
  const int DD = D * D;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  const int h = blockIdx.y;
  if (idx >= DD + D) return;
  const float* part = a.spart + static_cast<size_t>(h) * a.nsplit * (DD + D) + idx;
  // partials are fetched four at a time (independent loads in flight); the sum order stays fixed
  float add = 0.f;
  for (int s0 = 0; s0 < a.nsplit; s0 += 4) {
    float v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      v[i] = (s0 + i < a.nsplit) ? part[static_cast<size_t>(s0 + i) * (DD + D)] : 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) add += v[i];
  }
  if (idx < DD) {
    const size_t o = static_cast<size_t>(h) * DD + idx;
    const float s_old = a.S[o];
    const float s_new = s_old + add;
    a.S_prev[o] = s_old;
    a.S[o] = s_new;
    __nv_bfloat16* hl = a.hilo + static_cast<size_t>(h) * 4 * DD + idx;
    const __nv_bfloat16 nh = __float2bfloat16_rn(s_new);
    const __nv_bfloat16 oh = __float2bfloat16_rn(s_old);
    hl[0 * DD] = nh;
    hl[1 * DD] = __float2bfloat16_rn(s_new - __bfloat162float(nh));
    hl[2 * DD] = oh;
    hl[3 * DD] = __float2bfloat16_rn(s_old - __bfloat162float(oh));
  } else {
    const size_t o = static_cast<size_t>(h) * D + (idx - DD);
    const float z_old = a.z[o];
    a.z_prev[o] = z_old;
    a.z[o] = z_old + add;
  }
}

// ---------------------------------------------------------------------------------------
// Fused append for head_dim 128 (the measured path): one pass over the chunk's K and V.
// grid (nsplit, H); a CTA owns a run of consecutive history blocks of one head and, per block,
//   * copies the new rows into the block's page (and zero-fills the rest of a partial tail page),
//   * adds their column sums to the block's key sum,
//   * stages phi(K) (as bf16 hi + lo, so that hi + lo carries ~16 bits) and V in shared memory in
//     the 128-byte-swizzled MN-major layout and lets the tensor cores accumulate
//       S_part (128 x 128, fp32 in TMEM) += phi(K)_hi^T V + phi(K)_lo^T V
//     over the block's tokens (tcgen05, K = tokens), double-buffered against the next block's
//     loads,
// and finally writes its partial S and partial z for the fixed-order reduction of stage C.
// ---------------------------------------------------------------------------------------
namespace {

constexpr int kAfThreads = 512;
constexpr int kAfRowGroups = kAfThreads / 16;   // 32: a thread handles rows rg and rg + 32 of a block
constexpr int kAfRows = kBlock / kAfRowGroups;  // 2 rows per thread and block
constexpr int kAfTile = 64 * 128 * 2;           // [64 tokens x 128 dims] bf16 = two swizzled slabs
constexpr int kAfStage = 3 * kAfTile;           // phi hi | phi lo | V
constexpr int kAfRed = kAfRowGroups * 128 * 4;  // key-sum partials of one block
constexpr int kAfSmem = 2 * kAfStage + 2 * kAfRed + 64 + 1024;

struct AfBars {
  uint64_t mma_done[2];
  uint64_t all_done;
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
__device__ __forceinline__ float phi_fast(float x) { return x > 0.f ? x + 1.f : __expf(x); }

}  // namespace

__global__ void __launch_bounds__(kAfThreads, 1) append_fused_kernel(AppendArgs a, int blocks_per_cta) {
  constexpr int D = 128;
  extern __shared__ uint8_t af_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(af_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  float* red = reinterpret_cast<float*>(smem + 2 * kAfStage);  // [2][row groups][128]
  AfBars* bars = reinterpret_cast<AfBars*>(smem + 2 * kAfStage + 2 * kAfRed);

  const int h = blockIdx.y, split = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ch = threadIdx.x & 15;  // 16-byte chunk of a row (8 dims)
  const int rg = threadIdx.x >> 4;  // row group
  const int64_t b_first = a.n0 / kBlock, b_last = (a.n0 + a.n_new - 1) / kBlock;
  const int64_t bs = b_first + static_cast<int64_t>(split) * blocks_per_cta;
  const int64_t be = min64(b_last + 1, bs + blocks_per_cta);
  const int nblk = static_cast<int>(max64(0, be - bs));
  const int64_t n_end = a.n0 + a.n_new;

  if (threadIdx.x == 0) {
    mbar_init(&bars->mma_done[0], 1);
    mbar_init(&bars->mma_done[1], 1);
    mbar_init(&bars->all_done, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&bars->tmem_base, 128);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  uint4 kreg[kAfRows], vreg[kAfRows];
  auto load_block = [&](int64_t b, uint4 (&kk)[kAfRows], uint4 (&vv)[kAfRows]) {
#pragma unroll
    for (int i = 0; i < kAfRows; ++i) {
      const int64_t t = b * kBlock + rg + kAfRowGroups * i;
      if (t >= a.n0 && t < n_end) {
        const size_t src = static_cast<size_t>(t - a.n0) * a.tok_stride +
                           static_cast<size_t>(h) * a.head_stride + ch * 8;
        kk[i] = *reinterpret_cast<const uint4*>(a.k + src);
        vv[i] = *reinterpret_cast<const uint4*>(a.v + src);
      } else {
        kk[i] = make_uint4(0, 0, 0, 0);
        vv[i] = make_uint4(0, 0, 0, 0);
      }
    }
  };
  if (nblk > 0) load_block(bs, kreg, vreg);

  float zacc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) zacc[e] = 0.f;
  bool ok = true;

#pragma unroll 1
  for (int bi = 0; bi < nblk; ++bi) {
    const int64_t b = bs + bi;
    const int stage = bi & 1;
    uint8_t* st_hi = smem + stage * kAfStage;
    uint8_t* st_lo = st_hi + kAfTile;
    uint8_t* st_v = st_lo + kAfTile;
    float* my_red = red + stage * (kAfRowGroups * 128);
    uint4 knext[kAfRows], vnext[kAfRows];
    if (bi + 1 < nblk) load_block(b + 1, knext, vnext);  // next block's loads fly under this one
    // the tensor cores must be done with this stage's previous tiles (block bi - 2)
    if (bi >= 2) ok = af_wait(&bars->mma_done[stage], ((bi >> 1) - 1) & 1, bars, a.status) && ok;
    const int page = a.page_table[b];
    const size_t row_base = (static_cast<size_t>(page) * a.H + h) * kBlock;
    float ks[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) ks[e] = 0.f;
#pragma unroll
    for (int i = 0; i < kAfRows; ++i) {
      const int r = rg + kAfRowGroups * i;
      const int64_t t = b * kBlock + r;
      const bool fresh = t >= a.n0 && t < n_end;
      const uint32_t soff = (ch >> 3) * (kAfTile / 2) + r * 128 + (((ch & 7) ^ (r & 7)) << 4);
      // rows that are not new carry zeros (loaded as zeros above): they add nothing anywhere
      const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&kreg[i]);
      uint32_t hw[4], lw[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 f = __bfloat1622float2(k2[e]);
        ks[2 * e] += f.x;
        ks[2 * e + 1] += f.y;
        const float p0 = fresh ? phi_fast(f.x) : 0.f, p1 = fresh ? phi_fast(f.y) : 0.f;
        zacc[2 * e] += p0;
        zacc[2 * e + 1] += p1;
        const __nv_bfloat162 hh = __floats2bfloat162_rn(p0, p1);
        const float2 hf = __bfloat1622float2(hh);
        const __nv_bfloat162 ll = __floats2bfloat162_rn(p0 - hf.x, p1 - hf.y);
        hw[e] = *reinterpret_cast<const uint32_t*>(&hh);
        lw[e] = *reinterpret_cast<const uint32_t*>(&ll);
      }
      if (fresh || t >= n_end) {
        // new rows go to the page; rows of a partial tail page past the last token are zeroed so
        // that the pool never holds garbage the forward kernel could multiply by zero
        const size_t dst = (row_base + r) * D + ch * 8;
        *reinterpret_cast<uint4*>(a.k_pool + dst) = kreg[i];
        *reinterpret_cast<uint4*>(a.v_pool + dst) = vreg[i];
      }
      *reinterpret_cast<uint4*>(st_hi + soff) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
      *reinterpret_cast<uint4*>(st_lo + soff) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
      *reinterpret_cast<uint4*>(st_v + soff) = vreg[i];
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) my_red[rg * 128 + ch * 8 + e] = ks[e];
    fence_proxy_async_smem();  // generic-proxy writes above -> visible to the tensor cores
    __syncthreads();
    if (warp == 0) {
      if (elect_one_sync() && ok) {
        tc_fence_after();
        constexpr uint32_t idesc = idesc_bf16_f32(128, 128, 1, 1);
        constexpr uint32_t hi = desc_hi_sw128(1024);
        const uint32_t a_hi = desc_lo_sw128(smem_u32(st_hi), kAfTile / 2);
        const uint32_t a_lo = desc_lo_sw128(smem_u32(st_lo), kAfTile / 2);
        const uint32_t b_v = desc_lo_sw128(smem_u32(st_v), kAfTile / 2);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_ss_lo(tmem, a_hi + kk * 128, b_v + kk * 128, hi, idesc, (bi > 0 || kk > 0) ? 1u : 0u);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) tc_mma_ss_lo(tmem, a_lo + kk * 128, b_v + kk * 128, hi, idesc, 1u);
        tc_commit(&bars->mma_done[stage]);
      }
    } else if (threadIdx.x >= kAfThreads - 128) {
      // key sum of the block: fixed-order sum over the row groups
      const int c = threadIdx.x - (kAfThreads - 128);
      float s = 0.f;
#pragma unroll
      for (int g2 = 0; g2 < kAfRowGroups; ++g2) s += my_red[g2 * 128 + c];
      float* dst = a.ksum + (static_cast<size_t>(h) * a.max_pages + b) * D + c;
      const float old = (a.n0 > b * kBlock) ? *dst : 0.f;  // block partly filled before
      *dst = old + s;
    }
#pragma unroll
    for (int i = 0; i < kAfRows; ++i) {
      kreg[i] = knext[i];
      vreg[i] = vnext[i];
    }
  }

  // all tensor-core work of this CTA done?
  if (warp == 0) {
    if (elect_one_sync()) tc_commit(&bars->all_done);
  }
  ok = af_wait(&bars->all_done, 0, bars, a.status) && ok;
  tc_fence_after();
  float* out = a.spart + (static_cast<size_t>(h) * a.nsplit + split) * (D * D + D);
  {
    const int quad = warp & 3, part = warp >> 2;  // 16 warps: 4 lane quadrants x 4 column quarters
    const int row = quad * 32 + lane;
    uint32_t v[32];
    if (nblk > 0) {
      tmem_ld32(tmem + (static_cast<uint32_t>(quad * 32) << 16) + part * 32, v);
      tc_wait_ld();
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = 0u;
    }
    float4* dst = reinterpret_cast<float4*>(out + row * D + part * 32);
#pragma unroll
    for (int i = 0; i < 8; ++i)
      dst[i] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                           __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
  }
  // z partial: fixed-order sum over the row groups
  __syncthreads();
#pragma unroll
  for (int e = 0; e < 8; ++e) red[rg * 128 + ch * 8 + e] = zacc[e];
  __syncthreads();
  if (threadIdx.x < 128) {
    float s = 0.f;
#pragma unroll
    for (int g2 = 0; g2 < kAfRowGroups; ++g2) s += red[g2 * 128 + threadIdx.x];
    out[D * D + threadIdx.x] = s;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, 128);
  }
}

cudaError_t append_init() {
  return cudaFuncSetAttribute(append_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAfSmem);
}

cudaError_t launch_append(const AppendArgs& a_in, cudaStream_t st) {
  AppendArgs a = a_in;
  const int64_t b0 = a.n0 / kBlock;
  const int64_t b1 = (a.n0 + a.n_new - 1) / kBlock;
  cudaError_t e;
  if (a.D == 128 && a.lin_state) {
    const int nb = static_cast<int>(b1 - b0 + 1);
    const int per = (nb + a.nsplit - 1) / a.nsplit;
    a.nsplit = (nb + per - 1) / per;  // no empty CTAs
    dim3 grid(a.nsplit, a.H);
    append_fused_kernel<<<grid, kAfThreads, kAfSmem, st>>>(a, per);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  } else {
    dim3 gridA(static_cast<unsigned>(b1 - b0 + 1), a.H);
    if (a.D == 128)
      append_pool_ksum_kernel<128><<<gridA, 256, 0, st>>>(a);
    else
      append_pool_ksum_kernel<64><<<gridA, 256, 0, st>>>(a);
    e = cudaGetLastError();
    if (e != cudaSuccess || !a.lin_state) return e;
    dim3 gridB(a.nsplit, a.H);
    if (a.D == 128)
      state_partial_kernel<128><<<gridB, 256, 0, st>>>(a);
    else
      state_partial_kernel<64><<<gridB, 256, 0, st>>>(a);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  const int n = a.D * a.D + a.D;
  dim3 gridC((n + 255) / 256, a.H);
  state_reduce_kernel<<<gridC, 256, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace hsa
