// hsa_append_kv kernels: pool write + per-block key sums, and the linear-branch state update
//   S[h] += sum_j phi(k_j)^T v_j,   z[h] += sum_j phi(k_j),   phi(x) = elu(x) + 1
// as a deterministic two-stage reduction (no floating-point atomics).
#include <cuda_bf16.h>

#include "hsa_internal.h"

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
  float add = 0.f;
  for (int s = 0; s < a.nsplit; ++s) add += part[static_cast<size_t>(s) * (DD + D)];
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

cudaError_t launch_append(const AppendArgs& a, cudaStream_t st) {
  const int64_t b0 = a.n0 / kBlock;
  const int64_t b1 = (a.n0 + a.n_new - 1) / kBlock;
  dim3 gridA(static_cast<unsigned>(b1 - b0 + 1), a.H);
  if (a.D == 128)
    append_pool_ksum_kernel<128><<<gridA, 256, 0, st>>>(a);
  else
    append_pool_ksum_kernel<64><<<gridA, 256, 0, st>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess || !a.lin_state) return e;
  dim3 gridB(a.nsplit, a.H);
  if (a.D == 128)
    state_partial_kernel<128><<<gridB, 256, 0, st>>>(a);
  else
    state_partial_kernel<64><<<gridB, 256, 0, st>>>(a);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int n = a.D * a.D + a.D;
  dim3 gridC((n + 255) / 256, a.H);
  state_reduce_kernel<<<gridC, 256, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace hsa
