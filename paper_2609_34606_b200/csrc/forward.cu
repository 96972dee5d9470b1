// hsa_forward kernel for sm_100a.
//
// One CTA per (128-row query tile, head), 384 threads in three warpgroups:
//   warp 0       TMA producer: Q tile, then the selected K/V pages gathered through the page
//                table (two 64-token pages = 128 keys per step) into a 3-stage ring, then the
//                hi/lo halves of the linear state; also owns the TMEM allocation
//   warp 1       tcgen05.mma issuer: S = Q K^T, O += P V with P read from TMEM, then the linear
//                numerator phi(Q) S
//   warps 4..7   softmax group A: the even KV steps     } one query row per thread; each group
//   warps 8..11  softmax group B: the odd KV steps      } keeps its own running max / sum and
//                                                         its own O accumulator in TMEM
// The two groups never talk during the loop: while one exponentiates step j the tensor cores run
// Q K^T of a later step and P V of the other group's step.  The two partial results of a row
// are merged (log-sum-exp) in the epilogue, which also applies the linear branch and the gates
// and stores bf16 once.  TMEM: S_A | S_B | O_A | O_B (128 fp32 columns each); P overwrites the
// first 64 columns of its S buffer as packed bf16.
// Every barrier wait is bounded; when one gives up the kernel records a timeout in the status
// word and all roles drain to the common exit.
#include <cuda_bf16.h>

#include "hsa_internal.h"
#include "ptx.cuh"

namespace hsa {

namespace {

constexpr int kThreads = 384;
constexpr int kStages = 3;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;      // + 128 * group
constexpr uint32_t kColO = 256;    // + 128 * group
constexpr uint32_t kColLin = 0;    // linear numerator accumulator (after the loop)
constexpr uint32_t kColPhi = 128;  // phi(Q) as a bf16 A operand (after the loop)

template <int D>
struct Smem {
  static constexpr int kHalf = 128 * 128;    // bytes of one [128 rows x 128 B] slab
  static constexpr int kTile = 128 * D * 2;  // Q tile, K stage, V stage
  static constexpr int kQ = 0;
  static constexpr int kK = kTile;
  static constexpr int kV = kTile + kStages * kTile;
  static constexpr int kStats = kK;  // float[2][128][4], reuses K stage 0 once the loop is over
  static constexpr int kBars = kTile + 2 * kStages * kTile;
  static constexpr int kTotal = kBars + 256 + 1024;  // + alignment slack
};

struct Bars {
  uint64_t q_full;
  uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  uint64_t s_full[2];
  uint64_t p_full[2];
  uint64_t o_done;
  uint64_t lin_a_full;
  uint64_t lin_done;
  uint32_t tmem_base;
  volatile int abort_flag;
};

__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded barrier wait (about two seconds, or until another role has aborted).
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, Bars* bars,
                                         int32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = globaltimer_ns();
  for (uint32_t i = 1;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 0u) {
      if (bars->abort_flag) return false;
      if (globaltimer_ns() - t0 > 2000000000ull) {
        bars->abort_flag = 1;
        atomicCAS(status, 0, kDevTimeout);
        return false;
      }
    }
  }
}

#ifdef HSA_TIMING
__device__ long long g_hsa_timing[4096];
#define HSA_T(slot)                                                                  \
  do {                                                                               \
    if (blockIdx.x == 0 && blockIdx.y == 0 && lane == 0 && (slot) < 4096)             \
      g_hsa_timing[(slot)] = clock64();                                              \
  } while (0)
#else
#define HSA_T(slot) do { } while (0)
#endif

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float m;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(m) : "f"(a), "f"(b), "f"(c));
  return m;
}
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
// (a0, a1) * s2 + t2 on the packed fp32 pipe
__device__ __forceinline__ void ffma2(float& d0, float& d1, float a0, float a1, uint64_t s2,
                                      uint64_t t2) {
  uint64_t d;
  const uint64_t a = pack2(a0, a1);
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(s2), "l"(t2));
  asm("mov.b64 {%0, %1}, %2;" : "=f"(d0), "=f"(d1) : "l"(d));
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

}  // namespace

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
hsa_forward_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v,
                   const __grid_constant__ CUtensorMap tm_state, const FwdParams p) {
  using L = Smem<D>;
  constexpr int DH = D / 64;  // 64-element (128-byte) slabs per row
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  Bars* bars = reinterpret_cast<Bars*>(smem + L::kBars);
  float* stats = reinterpret_cast<float*>(smem + L::kStats);  // [group][row][m, l, den, -]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp == 4) HSA_T(3000);
  const int tile = blockIdx.x, h = blockIdx.y;
  const int row0 = tile * kTileM;
  const int g = p.group_tokens > 0 ? row0 / p.group_tokens : 0;
  const int32_t* sel = p.sel_idx + (static_cast<size_t>(h) * p.n_groups + g) * p.kcap;
  int cnt = p.do_sparse ? p.sel_cnt[static_cast<size_t>(h) * p.n_groups + g] : 0;
  cnt = max(0, min(cnt, p.kcap));
  const int nsteps = (cnt + 1) / 2;

  if (threadIdx.x == 0) {
    mbar_init(&bars->q_full, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->k_full[s], 1);
      mbar_init(&bars->k_empty[s], 1);
      mbar_init(&bars->v_full[s], 1);
      mbar_init(&bars->v_empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->s_full[i], 1);
      mbar_init(&bars->p_full[i], 128);
    }
    mbar_init(&bars->o_done, 1);
    mbar_init(&bars->lin_a_full, 256);
    mbar_init(&bars->lin_done, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&bars->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  if (warp == 4) HSA_T(3001);

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    if (warp == 0) {
      // ================================================================= TMA producer
      if (elect_one_sync()) {
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        mbar_expect_tx(&bars->q_full, L::kTile);
        for (int dh = 0; dh < DH; ++dh)
          tma_load_3d(smem + L::kQ + dh * L::kHalf, &tm_q, &bars->q_full, dh * 64, h, row0);
        bool ok = true;
        int armed_k = 0, armed_v = 0;  // loads issued per ring, for the drain on abort
#pragma unroll 1
        for (int j = 0; j < nsteps && ok; ++j) {
          const int s = j % kStages;
          const uint32_t ph = (j / kStages) & 1;
          const int npg = min(2, cnt - 2 * j);
          int32_t ycoord[2];
          for (int pg = 0; pg < npg; ++pg) {
            int blk = sel[2 * j + pg];
            if (blk < 0 || blk >= p.n_blocks) {  // never follow a bad index into the pool
              atomicCAS(p.status, 0, kDevBounds);
              blk = 0;
            }
            ycoord[pg] = (p.page_table[blk] * p.H + h) * kBlock;
          }
          ok = wait_bar(&bars->k_empty[s], ph ^ 1, bars, p.status);
          if (!ok) break;
          mbar_expect_tx(&bars->k_full[s], npg * kBlock * D * 2);
          for (int pg = 0; pg < npg; ++pg)
            for (int dh = 0; dh < DH; ++dh)
              tma_load_2d(smem + L::kK + s * L::kTile + dh * L::kHalf + pg * (kBlock * 128), &tm_k,
                          &bars->k_full[s], dh * 64, ycoord[pg]);
          ++armed_k;
          ok = wait_bar(&bars->v_empty[s], ph ^ 1, bars, p.status);
          if (!ok) break;
          mbar_expect_tx(&bars->v_full[s], npg * kBlock * D * 2);
          for (int pg = 0; pg < npg; ++pg)
            for (int dh = 0; dh < DH; ++dh)
              tma_load_2d(smem + L::kV + s * L::kTile + dh * L::kHalf + pg * (kBlock * 128), &tm_v,
                          &bars->v_full[s], dh * 64, ycoord[pg]);
          ++armed_v;
        }
        if (ok && p.do_linear) {
          // hi and lo halves of the D x D state ride the V ring as two more "steps"
          for (int hl = 0; hl < 2 && ok; ++hl) {
            const int j = nsteps + hl;
            const int s = j % kStages;
            const uint32_t ph = (j / kStages) & 1;
            ok = wait_bar(&bars->v_empty[s], ph ^ 1, bars, p.status);
            if (!ok) break;
            const int rbase = ((h * 2 + p.use_prev) * 2 + hl) * D;
            mbar_expect_tx(&bars->v_full[s], D * D * 2);
            for (int kb = 0; kb < DH; ++kb)
              for (int dh = 0; dh < DH; ++dh)
                tma_load_2d(smem + L::kV + s * L::kTile + dh * L::kHalf + kb * (kBlock * 128),
                            &tm_state, &bars->v_full[s], dh * 64, rbase + kb * 64);
            ++armed_v;
          }
        }
        if (!ok) {
          // drain: let every copy already issued land before the CTA's shared memory goes away
          for (int s = 0; s < kStages; ++s) {
            for (int i = 0; i < 2; ++i) {
              const int arms = i == 0 ? armed_k : armed_v;
              uint64_t* bar = i == 0 ? &bars->k_full[s] : &bars->v_full[s];
              const int last = ((arms - 1 - s) / kStages) * kStages + s;  // last step armed on s
              if (arms > s) mbar_wait(bar, (last / kStages) & 1, 1u << 16);
            }
          }
        }
      }
    } else if (warp == 1) {
      // ================================================================= MMA issuer
      if (elect_one_sync()) {
        constexpr uint32_t kHiSw = desc_hi_sw128(1024);
        const uint32_t q_lo = desc_lo_sw128(smem_u32(smem + L::kQ), 16);
        bool ok = wait_bar(&bars->q_full, 0, bars, p.status);
        tc_fence_after();
        HSA_T(3011);
        auto issue_qk = [&](int j) -> bool {
          const int s = j % kStages;
          if (!wait_bar(&bars->k_full[s], (j / kStages) & 1, bars, p.status)) return false;
          tc_fence_after();
          const uint32_t k_lo = desc_lo_sw128(smem_u32(smem + L::kK + s * L::kTile), 16);
          const uint32_t d_tmem = tmem + kColS + 128 * (j & 1);
          if (cnt - 2 * j >= 2) {
            constexpr uint32_t idesc = idesc_bf16_f32(128, 128, 0, 0);
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t off = ((kk / 4) * L::kHalf + (kk % 4) * 32) >> 4;
              tc_mma_ss_lo(d_tmem, q_lo + off, k_lo + off, kHiSw, idesc, kk > 0 ? 1u : 0u);
            }
          } else {
            constexpr uint32_t idesc = idesc_bf16_f32(128, 64, 0, 0);
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t off = ((kk / 4) * L::kHalf + (kk % 4) * 32) >> 4;
              tc_mma_ss_lo(d_tmem, q_lo + off, k_lo + off, kHiSw, idesc, kk > 0 ? 1u : 0u);
            }
          }
          tc_commit(&bars->k_empty[s]);
          tc_commit(&bars->s_full[j & 1]);
          return true;
        };
        if (ok && nsteps > 0) ok = issue_qk(0);
        if (ok && nsteps > 1) ok = issue_qk(1);
#pragma unroll 1
        for (int j = 0; j < nsteps && ok; ++j) {
          const int s = j % kStages;
          HSA_T(2048 + j * 8 + 0);
          ok = wait_bar(&bars->p_full[j & 1], (j >> 1) & 1, bars, p.status);
          if (!ok) break;
          HSA_T(2048 + j * 8 + 1);
          ok = wait_bar(&bars->v_full[s], (j / kStages) & 1, bars, p.status);
          if (!ok) break;
          tc_fence_after();
          HSA_T(2048 + j * 8 + 2);
          constexpr uint32_t idesc = idesc_bf16_f32(128, D, 0, 1);
          const uint32_t v_lo = desc_lo_sw128(smem_u32(smem + L::kV + s * L::kTile), L::kHalf);
          const uint32_t o_acc = tmem + kColO + 128 * (j & 1);
          const uint32_t p_op = tmem + kColS + 128 * (j & 1);
          const uint32_t acc0 = j >= 2 ? 1u : 0u;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            tc_mma_ts_lo(o_acc, p_op + kk * 8, v_lo + kk * 128, kHiSw, idesc, kk > 0 ? 1u : acc0);
          if (cnt - 2 * j >= 2) {
#pragma unroll
            for (int kk = 4; kk < 8; ++kk)
              tc_mma_ts_lo(o_acc, p_op + kk * 8, v_lo + kk * 128, kHiSw, idesc, 1u);
          }
          tc_commit(&bars->v_empty[s]);
          HSA_T(2048 + j * 8 + 3);
          // the next scores of this group overwrite the P just consumed: issued after the P V
          // above, the tensor pipe runs them in order
          if (j + 2 < nsteps) ok = issue_qk(j + 2);
          HSA_T(2048 + j * 8 + 4);
        }
        if (ok) tc_commit(&bars->o_done);
        if (ok && p.do_linear) {
          ok = wait_bar(&bars->lin_a_full, 0, bars, p.status);
          for (int hl = 0; hl < 2 && ok; ++hl) {
            const int j = nsteps + hl;
            const int s = j % kStages;
            ok = wait_bar(&bars->v_full[s], (j / kStages) & 1, bars, p.status);
            if (!ok) break;
            tc_fence_after();
            constexpr uint32_t idesc = idesc_bf16_f32(128, D, 0, 1);
            const uint32_t b_lo = desc_lo_sw128(smem_u32(smem + L::kV + s * L::kTile), L::kHalf);
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk)
              tc_mma_ts_lo(tmem + kColLin, tmem + kColPhi + kk * 8, b_lo + kk * 128, kHiSw, idesc,
                           (hl > 0 || kk > 0) ? 1u : 0u);
            tc_commit(&bars->v_empty[s]);
          }
          if (ok) tc_commit(&bars->lin_done);
        }
      }
    }
  } else {
    // ================================================================= softmax groups + epilogue
    asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
    const int grp = (warp - 4) >> 2;                 // 0: even steps, 1: odd steps
    const int quad = warp & 3;                       // TMEM lane quadrant this warp may access
    const int r = quad * 32 + lane;                  // row inside the tile
    const int row = row0 + r;                        // query index inside the chunk
    const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
    const uint32_t s_tmem = tmem + lane_off + kColS + 128 * grp;
    const uint32_t o_tmem = tmem + lane_off + kColO + 128 * grp;
    const int64_t qpos = p.q_pos0 + row;
    const int64_t vis_end = p.causal ? min64(p.n_tokens, qpos + 1) : p.n_tokens;
    // the first row of the tile sees the fewest keys: a step whose pages all end at or before
    // that row's limit needs no masking
    const int64_t tile_vis_end = p.causal ? min64(p.n_tokens, p.q_pos0 + row0 + 1) : p.n_tokens;
    const float sl2 = p.scale_log2;
    float m_used = -INFINITY;  // reference maximum the stored exponents are relative to (raw)
    float l = 0.f;
    bool ok = true;

    // block ids of this group's next step are fetched one step ahead, off the critical path
    int nb0 = 0, nb1 = 0;
    if (grp < nsteps) {
      nb0 = sel[2 * grp];
      nb1 = (2 * grp + 1 < cnt) ? sel[2 * grp + 1] : 0;
    }
#pragma unroll 1
    for (int j = grp; j < nsteps; j += 2) {
      int blk0 = nb0, blk1 = nb1;
      if (j + 2 < nsteps) {
        nb0 = sel[2 * (j + 2)];
        nb1 = (2 * (j + 2) + 1 < cnt) ? sel[2 * (j + 2) + 1] : 0;
      }
      if (quad == 0) HSA_T(grp * 1024 + (j >> 1) * 8 + 0);
      ok = __all_sync(0xffffffffu, wait_bar(&bars->s_full[grp], (j >> 1) & 1, bars, p.status));
      if (!ok) break;
      tc_fence_after();
      if (quad == 0) HSA_T(grp * 1024 + (j >> 1) * 8 + 1);
      const int npg = min(2, cnt - 2 * j);
      const int n = npg * kBlock;
      uint32_t sr[128];
      tmem_ld32(s_tmem + 0, reinterpret_cast<uint32_t(&)[32]>(sr[0]));
      tmem_ld32(s_tmem + 32, reinterpret_cast<uint32_t(&)[32]>(sr[32]));
      if (n == 128) {
        tmem_ld32(s_tmem + 64, reinterpret_cast<uint32_t(&)[32]>(sr[64]));
        tmem_ld32(s_tmem + 96, reinterpret_cast<uint32_t(&)[32]>(sr[96]));
      }
      if (blk0 < 0 || blk0 >= p.n_blocks) blk0 = 0;
      if (blk1 < 0 || blk1 >= p.n_blocks) blk1 = 0;
      const int64_t last_blk = blk0 > blk1 ? blk0 : blk1;
      const bool need_mask = (n != 128) || (last_blk * kBlock + kBlock > tile_vis_end);
      tc_wait_ld();
      if (quad == 0) HSA_T(grp * 1024 + (j >> 1) * 8 + 2);
      if (need_mask) {
        // visible keys per page: columns [0, lim) of the page's 64
        const int lim0 = static_cast<int>(max64(0, min64(kBlock, vis_end - static_cast<int64_t>(blk0) * kBlock)));
        const int lim1 =
            npg > 1 ? static_cast<int>(max64(0, min64(kBlock, vis_end - static_cast<int64_t>(blk1) * kBlock))) : 0;
#pragma unroll
        for (int c = 0; c < 128; ++c) {
          const bool valid = (c & 63) < ((c >> 6) ? lim1 : lim0);
          if (!valid) sr[c] = 0xff800000u;  // -inf
        }
      }
      // row maximum: four independent chains
      float mx[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) mx[q] = fmaxf(__uint_as_float(sr[32 * q]), __uint_as_float(sr[32 * q + 1]));
#pragma unroll
      for (int c = 2; c < 32; c += 2)
#pragma unroll
        for (int q = 0; q < 4; ++q)
          mx[q] = fmax3(mx[q], __uint_as_float(sr[32 * q + c]), __uint_as_float(sr[32 * q + c + 1]));
      const float m_new = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
      if (quad == 0) HSA_T(grp * 1024 + (j >> 1) * 8 + 3);
      // lazy rescale: move the reference maximum only when it would grow by more than 2^8
      float factor = 1.f;
      if (m_used == -INFINITY) {
        m_used = m_new;  // nothing accumulated so far (O and l are zero or not yet written)
      } else if ((m_new - m_used) * sl2 > 8.f) {
        factor = ex2((m_used - m_new) * sl2);
        l *= factor;
        m_used = m_new;
      }
      // O of this group is quiescent here: its previous P V completed before this step's scores
      // were committed, and its next P V waits for the P written below
      if (j >= 2 && __any_sync(0xffffffffu, factor != 1.f)) {
#pragma unroll 1
        for (int c0 = 0; c0 < D; c0 += 32) {
          uint32_t o[32];
          tmem_ld32(o_tmem + c0, o);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
          tmem_st32(o_tmem + c0, o);
        }
      }
      const float moff = (m_used == -INFINITY) ? 0.f : m_used * sl2;
      const uint64_t s2 = pack2(sl2, sl2), t2 = pack2(-moff, -moff);
      uint64_t acc0 = 0, acc1 = 0;  // two packed fp32 pairs of partial row sums
#pragma unroll
      for (int c = 0; c < 128; c += 4) {
        float x0, x1, x2, x3;
        ffma2(x0, x1, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]), s2, t2);
        ffma2(x2, x3, __uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3]), s2, t2);
        const float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);
        acc0 = fadd2(acc0, pack2(p0, p1));
        acc1 = fadd2(acc1, pack2(p2, p3));
        sr[c >> 1] = pack_bf16(p0, p1);
        sr[(c >> 1) + 1] = pack_bf16(p2, p3);
      }
      {
        float a, b, c2, d2;
        unpack2(acc0, a, b);
        unpack2(acc1, c2, d2);
        l += (a + b) + (c2 + d2);
      }
      if (quad == 0) HSA_T(grp * 1024 + (j >> 1) * 8 + 4);
      tmem_st32(s_tmem, reinterpret_cast<uint32_t(&)[32]>(sr[0]));
      if (n == 128) tmem_st32(s_tmem + 32, reinterpret_cast<uint32_t(&)[32]>(sr[32]));
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->p_full[grp]);
      if (quad == 0) HSA_T(grp * 1024 + (j >> 1) * 8 + 5);
    }

    // ---------------------------------------------------------------- epilogue
    if (ok && nsteps > 0) {
      ok = __all_sync(0xffffffffu, wait_bar(&bars->o_done, 0, bars, p.status));
      tc_fence_after();
    }
    if (quad == 0) HSA_T(3002 + grp);
    // this group's columns of the output row: group 0 -> [0, D/2), group 1 -> [D/2, D)
    constexpr int HC = D / 2;
    const int cbase = grp * HC;
    float den_part = 0.f;
    if (ok && p.do_linear) {
      // phi(q) of this thread's row for its half of the dims -> bf16 A operand in TMEM;
      // partial denominator phi(q) . z over the same dims
      ok = __all_sync(0xffffffffu, wait_bar(&bars->q_full, 0, bars, p.status));
      const uint8_t* qrow = smem + L::kQ + r * 128;
      const float4* z4 = reinterpret_cast<const float4*>(p.z + static_cast<size_t>(h) * D + cbase);
      uint32_t fr[HC / 2];
#pragma unroll
      for (int c16 = 0; c16 < HC / 8; ++c16) {
        const float4 za = z4[c16 * 2], zb = z4[c16 * 2 + 1];
        const float z[8] = {za.x, za.y, za.z, za.w, zb.x, zb.y, zb.z, zb.w};
        const int cc = cbase / 8 + c16;  // 16-byte chunk of the row
        const int dh = cc >> 3, ch = cc & 7;
        const uint4 raw = *reinterpret_cast<const uint4*>(qrow + dh * L::kHalf + ((ch ^ (r & 7)) << 4));
        const __nv_bfloat162* q2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __bfloat1622float2(q2[i]);
          const float a0 = f.x > 0.f ? f.x + 1.f : __expf(f.x);
          const float a1 = f.y > 0.f ? f.y + 1.f : __expf(f.y);
          const __nv_bfloat162 pk = __floats2bfloat162_rn(a0, a1);
          fr[c16 * 4 + i] = *reinterpret_cast<const uint32_t*>(&pk);
          const float2 rr = __bfloat1622float2(pk);  // the rounded values the MMA will see
          den_part = fmaf(rr.x, z[2 * i], den_part);
          den_part = fmaf(rr.y, z[2 * i + 1], den_part);
        }
      }
      if constexpr (D == 128) {
        tmem_st32(tmem + lane_off + kColPhi + grp * 32, reinterpret_cast<uint32_t(&)[32]>(fr[0]));
      } else {
        tmem_st16(tmem + lane_off + kColPhi + grp * 16, reinterpret_cast<uint32_t(&)[16]>(fr[0]));
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->lin_a_full);
    }
    // publish this group's row statistics, then read the other group's
    stats[(grp * 128 + r) * 4 + 0] = m_used;
    stats[(grp * 128 + r) * 4 + 1] = l;
    stats[(grp * 128 + r) * 4 + 2] = den_part;
    if (quad == 0) HSA_T(3004 + grp);
    named_bar_sync(1, 256);
    const float m_o = stats[((grp ^ 1) * 128 + r) * 4 + 0];
    const float l_o = stats[((grp ^ 1) * 128 + r) * 4 + 1];
    const float den = den_part + stats[((grp ^ 1) * 128 + r) * 4 + 2];
    // log-sum-exp merge of the two partial softmax results of this row
    const float mm = fmaxf(m_used, m_o);
    const float c_me = (m_used == -INFINITY) ? 0.f : ex2((m_used - mm) * sl2);
    const float c_ot = (m_o == -INFINITY) ? 0.f : ex2((m_o - mm) * sl2);
    const float lsum = l * c_me + l_o * c_ot;
    const float inv_l = lsum > 0.f ? 1.f / lsum : 0.f;
    const float w_a = (grp == 0 ? c_me : c_ot) * inv_l;  // weight of accumulator A
    const float w_b = (grp == 0 ? c_ot : c_me) * inv_l;  // weight of accumulator B
    const bool has_a = nsteps > 0, has_b = nsteps > 1;
    if (ok && p.do_linear) {
      ok = __all_sync(0xffffffffu, wait_bar(&bars->lin_done, 0, bars, p.status));
      tc_fence_after();
    }
    if (quad == 0) HSA_T(3006 + grp);
    if (ok) {  // warp-uniform: the TMEM loads below are warp-collective
      const bool wr = row < p.n_q;  // rows past the end of the chunk compute but never store
      float lin_den = den;
      const float* lnum = nullptr;
      if (wr && p.do_linear && p.lin_num != nullptr) {
        lnum = p.lin_num + (static_cast<size_t>(row) * p.H + h) * D;
        lin_den += p.lin_den[static_cast<size_t>(row) * p.H + h];
      }
      const float inv_den = (p.do_linear && lin_den > 0.f) ? 1.f / lin_den : 0.f;
      __nv_bfloat16* orow = p.out + static_cast<size_t>(row) * p.o_ts + static_cast<size_t>(h) * p.o_hs;
      const __nv_bfloat16* gl =
          (wr && p.g_lin) ? p.g_lin + static_cast<size_t>(row) * p.g_ts + static_cast<size_t>(h) * p.g_hs : nullptr;
      const __nv_bfloat16* gs =
          (wr && p.g_sp) ? p.g_sp + static_cast<size_t>(row) * p.g_ts + static_cast<size_t>(h) * p.g_hs : nullptr;
      const int g_ds = static_cast<int>(p.g_ds);
      const bool sig = p.gate_act == 1;
      // rolled on purpose: 16 columns per trip keeps this once-per-tile code small
#pragma unroll 1
      for (int c0 = cbase; c0 < cbase + HC; c0 += 16) {
        uint32_t oa[16], ob[16], ln[16];
        if (has_a) tmem_ld16(tmem + lane_off + kColO + c0, oa);
        if (has_b) tmem_ld16(tmem + lane_off + kColO + 128 + c0, ob);
        if (p.do_linear) tmem_ld16(tmem + lane_off + kColLin + c0, ln);
        tc_wait_ld();
        uint32_t packed[8];
#pragma unroll
        for (int i = 0; i < 16; i += 2) {
          float res[2];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            float osp = 0.f;
            if (has_a) osp = __uint_as_float(oa[i + e]) * w_a;
            if (has_b) osp = fmaf(__uint_as_float(ob[i + e]), w_b, osp);
            float olin = 0.f;
            if (p.do_linear) {
              float num = __uint_as_float(ln[i + e]);
              if (lnum) num += lnum[c0 + i + e];
              olin = num * inv_den;
            }
            if (gl) {
              float wl = __bfloat162float(gl[(c0 + i + e) * g_ds]);
              if (sig) wl = __fdividef(1.f, 1.f + __expf(-wl));
              olin *= wl;
            }
            if (gs) {
              float ws = __bfloat162float(gs[(c0 + i + e) * g_ds]);
              if (sig) ws = __fdividef(1.f, 1.f + __expf(-ws));
              osp *= ws;
            }
            res[e] = olin + osp;
          }
          packed[i >> 1] = pack_bf16(res[0], res[1]);
        }
        if (wr) {
          *reinterpret_cast<uint4*>(orow + c0) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
          *reinterpret_cast<uint4*>(orow + c0 + 8) = make_uint4(packed[4], packed[5], packed[6], packed[7]);
        }
      }
    }
  }

  if (warp == 4 || warp == 8) HSA_T(3008 + (warp == 8));
  // ------------------------------------------------------------------- common exit
  tc_fence_before();
  __syncthreads();
  if (warp == 4) HSA_T(3010);
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

#ifdef HSA_TIMING
extern "C" int hsa_debug_read_timing(long long* host_out, int n) {
  return static_cast<int>(cudaMemcpyFromSymbol(host_out, g_hsa_timing, sizeof(long long) * n));
}
#endif

cudaError_t forward_init() {
  cudaError_t e = cudaFuncSetAttribute(hsa_forward_kernel<128>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<128>::kTotal);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(hsa_forward_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Smem<64>::kTotal);
}

cudaError_t launch_forward(const FwdParams& p, int D, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                           const CUtensorMap& tm_v, const CUtensorMap& tm_state, cudaStream_t st) {
  const int n_tiles = (p.n_q + kTileM - 1) / kTileM;
  dim3 grid(n_tiles, p.H);
  if (D == 128)
    hsa_forward_kernel<128><<<grid, kThreads, Smem<128>::kTotal, st>>>(tm_q, tm_k, tm_v, tm_state, p);
  else
    hsa_forward_kernel<64><<<grid, kThreads, Smem<64>::kTotal, st>>>(tm_q, tm_k, tm_v, tm_state, p);
  return cudaGetLastError();
}

}  // namespace hsa
