// hsa_forward kernel for sm_100a.
//
// Work items are (128-row query tile, head) pairs.  The plain kernel is persistent: one CTA per SM
// takes the items b, b + gridDim.x, ... and the barriers, rings and score buffers run on from item
// to item, so that the Q tile, the first K steps and the first Q K^T of the next item are
// requested / issued under the epilogue of the current one.  The split kernel (long lists) has one
// CTA per (tile, head, part).  384 threads in three warpgroups:
//   warp 0       TMA producer: Q tile, then the selected K/V pages gathered through the page
//                table (two 64-token pages = 128 keys per step) into two 3-stage rings, then the
//                hi/lo halves of the linear state; also owns the TMEM allocation
//   warp 1       tcgen05.mma issuer: S = Q K^T three steps ahead, O += P V with P read from
//                TMEM, then the linear numerator phi(Q) S
//   warps 4..11  two softmax groups of four warps: group g takes the KV steps j = g (mod 2);
//                one query row per thread
// TMEM: O (128 fp32 columns) | three S buffers (128 columns each); P overwrites the first 64
// columns of its S buffer as packed bf16.  With three score buffers the tensor pipe never waits
// for a softmax group: Q K^T of step j+3 is issued right after P V of step j.
//
// Both groups accumulate into ONE O.  That needs a common exponent reference per row, so in the
// normal ("fast") pass the reference is fixed once: the row maximum of the first step plus a
// headroom of 2^20.  Every later weight is exp2(s - ref) with no running maximum and no rescale.
// fp32 / bf16 carry the same relative precision at any magnitude, so the result equals the
// usual online softmax as long as no weight overflows; a step whose weights exceed 2^27 sets a
// flag and the tile is redone in a "safe" pass: one group, classic online softmax with lazy
// rescale.  The two groups' partial row sums are added in the epilogue, which also applies the
// linear branch and the gates and stores bf16 once.
// Every barrier wait is bounded; when one gives up the kernel records a timeout in the status
// word and all roles drain to the common exit.
#include <cuda_bf16.h>

#include "hsa_internal.h"
#include "ptx.cuh"

namespace hsa {

namespace {

#ifndef HSA_GROUPS
#define HSA_GROUPS 2
#endif
#ifndef HSA_SMREGS
#define HSA_SMREGS 224
#endif
constexpr int kGroups = HSA_GROUPS;  // softmax groups; group g takes the KV steps j = g (mod kGroups)
constexpr bool kTokens = false;       // serialise the groups' exponential phases (2 groups only)
constexpr int kThreads = 128 + 128 * kGroups;
constexpr int kStages = 3;   // K ring and V ring depth
constexpr int kSBufs = 3;    // score buffers in TMEM
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColO = 0;
constexpr uint32_t kColS = 128;    // + 128 * buffer
constexpr uint32_t kColPhi = 128;  // phi(Q) as a bf16 A operand (after the loop: buffer 0)
constexpr uint32_t kColLin = 256;  // linear numerator accumulator (after the loop: buffer 1)
constexpr float kHeadroom = 20.f;  // log2 units below 1 at which the first step's maximum sits
constexpr float kRedoSum = 134217728.f;  // 2^27: a step's row sum above this forces the safe pass

template <int D>
struct Smem {
  static constexpr int kHalf = 128 * 128;    // bytes of one [128 rows x 128 B] slab
  static constexpr int kTile = 128 * D * 2;  // Q tile, K stage, V stage
  static constexpr int kQ = 0;
  static constexpr int kK = kTile;
  static constexpr int kV = kTile + kStages * kTile;
  static constexpr int kBars = kTile + 2 * kStages * kTile;
  static constexpr int kBarBytes = 3072;         // barriers and per-row values
  static constexpr int kTotal = kBars + kBarBytes;  // the dynamic shared memory must start on a 1 KB boundary
};

struct Bars {
  uint64_t q_full;
  int ticket;  // split tiles: arrival number of this CTA among the parts of its (tile, head)
  uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  uint64_t s_full[kSBufs];
  uint64_t p_full[kSBufs];
  uint64_t pv_done;
  uint64_t o_done;
  uint64_t mref_ready;
  uint64_t tok[2];  // exponential-phase token: the two softmax groups take turns on the SFU
  uint64_t lin_a_full;
  uint64_t lin_done;
  uint64_t final_known;  // the MMA lane has seen the last P of the item: `final` is valid
  uint64_t o_free;       // both groups have read the accumulators of the item out of TMEM
  uint32_t tmem_base;
  volatile int abort_flag;
  volatile int redo;
  volatile int final;    // this attempt's result stands (no safe pass follows)
  float mref[128];       // per-row exponent reference (log2 domain) of the fast pass
  float2 stat[2][128];   // per group and row: partial row sum, partial linear denominator
};
static_assert(sizeof(Bars) <= 3072, "barrier block must fit its shared-memory slot");

#ifndef HSA_INTERLEAVE
#define HSA_INTERLEAVE 8
#endif
#ifndef HSA_CONTINUOUS
#define HSA_CONTINUOUS 8
#endif
#ifdef HSA_TIMING
#ifndef HSA_T_BX
#define HSA_T_BX 0
#define HSA_T_BY 0
#endif
__device__ long long g_hsa_timing[4096];
#define HSA_T(slot)                                                      \
  do {                                                                   \
    if (blockIdx.x == HSA_T_BX && blockIdx.y == HSA_T_BY && lane == 0 && (slot) < 4096) \
      g_hsa_timing[(slot)] = clock64();                                  \
  } while (0)
#else
#define HSA_T(slot) \
  do {              \
  } while (0)
#endif

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

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// same, but ordered against the other volatile statements (keeps a hand-made instruction order)
__device__ __forceinline__ float ex2v(float x) {
  float y;
  asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// phi(x) = elu(x) + 1 = max(x, 0) + exp(min(x, 0))
__device__ __forceinline__ float phi_elu1(float x) {
  return fmaxf(x, 0.f) + ex2(fminf(x, 0.f) * 1.4426950408889634f);
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
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
// (a0, a1) * s2 + t2 on the packed fp32 pipe
__device__ __forceinline__ void ffma2(float& d0, float& d1, float a0, float a1, uint64_t s2,
                                      uint64_t t2) {
  uint64_t d;
  const uint64_t a = pack2(a0, a1);
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(s2), "l"(t2));
  unpack2(d, d0, d1);
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

__device__ __forceinline__ void init_barriers(Bars* bars) {
  mbar_init(&bars->q_full, 1);
  for (int s = 0; s < kStages; ++s) {
    mbar_init(&bars->k_full[s], 1);
    mbar_init(&bars->k_empty[s], 1);
    mbar_init(&bars->v_full[s], 1);
    mbar_init(&bars->v_empty[s], 1);
  }
  for (int i = 0; i < kSBufs; ++i) {
    mbar_init(&bars->s_full[i], 1);
    mbar_init(&bars->p_full[i], 128);
  }
  mbar_init(&bars->pv_done, 1);
  mbar_init(&bars->o_done, 1);
  mbar_init(&bars->mref_ready, 128);  // group 0 publishes the per-row reference
  mbar_init(&bars->tok[0], 128);
  mbar_init(&bars->tok[1], 128);
  mbar_init(&bars->lin_a_full, 256);
  mbar_init(&bars->lin_done, 1);
  mbar_init(&bars->final_known, 1);
  mbar_init(&bars->o_free, 128 * kGroups);
  bars->redo = 0;
  fence_mbar_init();
}

}  // namespace

// SPLIT: compiled with the split-tile path (grid z > 1); the plain kernel carries none of it
template <int D, bool SPLIT>
__global__ void __launch_bounds__(kThreads, 1)
hsa_forward_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v,
                   const __grid_constant__ CUtensorMap tm_state,
                   const __grid_constant__ CUtensorMap tm_out, const FwdParams p) {
  using L = Smem<D>;
  constexpr int DH = D / 64;  // 64-element (128-byte) slabs per row
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = smem_raw;
  Bars* bars = reinterpret_cast<Bars*>(smem + L::kBars);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp == 4) HSA_T(3000);
  if ((smem_u32(smem) & 1023u) != 0u) {  // the swizzled tiles need the 1 KB boundary
    if (threadIdx.x == 0) atomicCAS(p.status, 0, kDevBounds);
    return;
  }
  // Work items are (tile, head) pairs, tile fastest.  The plain kernel is persistent: CTA b takes the
  // items b, b + gridDim.x, ... one after the other, so that the set-up, the first loads and the
  // first Q K^T of an item run under the epilogue of the item before it.  The split kernel keeps
  // one item per CTA: grid (tile, head, part).
  const int n_tiles = (p.n_q + kTileM - 1) / kTileM;
  const int n_items = n_tiles * p.H;
  const int item0 = SPLIT ? static_cast<int>(blockIdx.y) * n_tiles + static_cast<int>(blockIdx.x) : static_cast<int>(blockIdx.x);
  const int item_stride = SPLIT ? n_items : static_cast<int>(gridDim.x);
  const int part = SPLIT ? static_cast<int>(blockIdx.z) : 0;
  const int nparts = SPLIT ? static_cast<int>(gridDim.z) : 1;
  struct Item {
    int tile, h, row0, cnt, nsteps, nsplit;
    const int32_t* sel;
  };
  auto get_item = [&](int item) -> Item {
    Item I;
    I.tile = item % n_tiles;
    I.h = item / n_tiles;
    I.row0 = I.tile * kTileM;
    const int g = p.group_tokens > 0 ? I.row0 / p.group_tokens : 0;
    I.sel = p.sel_idx + (static_cast<size_t>(I.h) * p.n_groups + g) * p.kcap;
    int cnt = p.do_sparse ? p.sel_cnt[static_cast<size_t>(I.h) * p.n_groups + g] : 0;
    cnt = max(0, min(cnt, min(p.kcap, p.n_blocks)));  // never more blocks than the history holds
    // A long list is split over the CTAs (tile, head, 0 .. nsplit - 1): each takes a run of whole
    // two-page steps; CTAs beyond nsplit leave before they set anything up.
    I.nsplit = 1;
    if (SPLIT && nparts > 1) {
      const int steps_total = (cnt + 1) / 2;
      const int split_steps = p.split_blocks / 2;
      int nsplit = min(nparts, max(1, (steps_total + split_steps - 1) / split_steps));
      const int steps_per = (steps_total + nsplit - 1) / nsplit;
      if (steps_per > 0) nsplit = (steps_total + steps_per - 1) / steps_per;  // no empty part
      I.nsplit = nsplit;
      if (nsplit > 1 && part < nsplit) {
        const int b_lo = 2 * part * steps_per;
        const int b_hi = min(cnt, 2 * (part + 1) * steps_per);
        I.sel += b_lo;
        cnt = b_hi - b_lo;
      }
    }
    I.cnt = cnt;
    I.nsteps = (cnt + 1) / 2;
    return I;
  };
  if (SPLIT && part >= get_item(item0).nsplit) return;

  if (threadIdx.x == 0) {
    bars->abort_flag = 0;
    init_barriers(bars);
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

  // attempt 0: fast pass (fixed exponent reference); attempt 1 only if a step overflowed: safe
  // pass.  Both role branches run the same attempt loop and meet at the same CTA-wide barriers.
  bool safe = false;
  auto end_of_attempt = [&]() -> bool {  // true: run the safe pass next
    tc_fence_before();
    __syncthreads();
    if (safe || bars->redo == 0 || bars->abort_flag) return false;
    // a fast-pass step overflowed its fixed reference: every barrier starts over
    __syncthreads();
    if (threadIdx.x == 0) {
      init_barriers(bars);
      atomicAdd(p.status + 1, 1);  // informational: tiles that needed the safe pass
    }
    __syncthreads();
    tc_fence_after();
    return true;
  };

  // Running counters, the same in every role: K / score steps and V steps (the state halves count
  // as two) since the barriers were last initialised, and items since then.  Ring stage, score
  // buffer and barrier parity of a step all follow from them, so the rings run on across items.
  int G = 0, Gv = 0, ic = 0;
  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    // one lane of warp 0 and one of warp 1 do the issuing; elected once, because they carry state
    // from item to item
    const bool leader = elect_one_sync();
    if (warp == 0 && leader) {
      tma_prefetch_desc(&tm_q);
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
    }
    // what the tail of the previous item has already done for this one (plain kernel only)
    int pre_k = -1;       // producer: Q requested and this many K steps; -1: nothing
    bool pre_qk = false;  // MMA lane: the first Q K^T are issued
#pragma unroll 1
    for (int item = item0; item < n_items; item += item_stride) {
    const Item I = get_item(item);
    const int h = I.h, row0 = I.row0, cnt = I.cnt, nsteps = I.nsteps;
    const int32_t* sel = I.sel;
    safe = false;
#pragma unroll 1
    for (int attempt = 0; attempt < 2; ++attempt) {
    if (warp == 0) {
      // ================================================================= TMA producer
      if (leader) {
        auto load_q = [&](int xh, int xrow0) {
          mbar_expect_tx(&bars->q_full, L::kTile);
          for (int dh = 0; dh < DH; ++dh)
            tma_load_3d(smem + L::kQ + dh * L::kHalf, &tm_q, &bars->q_full, dh * 64, xh, xrow0);
        };
        if (pre_k < 0) load_q(h, row0);
        bool ok = true;
        int armed_k = 0, armed_v = 0;  // loads issued per ring in this attempt, for the drain on abort
        // step j of the item (xsel, xcnt, xh), whose steps start at gbase in its ring
        auto load_kv = [&](const int32_t* xsel, int xcnt, int xh, int gbase, int j, bool is_k) -> bool {
          auto page_row = [&](int idx) -> int32_t {
            int blk = xsel[idx];
            if (blk < 0 || blk >= p.n_blocks) {  // never follow a bad index into the pool
              atomicCAS(p.status, 0, kDevBounds);
              blk = 0;
            }
            return (p.page_table[blk] * p.H + xh) * kBlock;
          };
          const int gj = gbase + j;
          const int s = gj % kStages;
          const uint32_t ph = (gj / kStages) & 1;
          const int npg = min(2, xcnt - 2 * j);
          uint64_t* full = is_k ? &bars->k_full[s] : &bars->v_full[s];
          uint64_t* empty = is_k ? &bars->k_empty[s] : &bars->v_empty[s];
          uint8_t* dst = smem + (is_k ? L::kK : L::kV) + s * L::kTile;
          const void* tm = is_k ? static_cast<const void*>(&tm_k) : static_cast<const void*>(&tm_v);
          int32_t y[2] = {0, 0};
          for (int pg = 0; pg < npg; ++pg) y[pg] = page_row(2 * j + pg);
          if (!wait_bar(empty, ph ^ 1, bars, p.status)) return false;
          mbar_expect_tx(full, npg * kBlock * D * 2);
          for (int pg = 0; pg < npg; ++pg)
            for (int dh = 0; dh < DH; ++dh)
              tma_load_2d(dst + dh * L::kHalf + pg * (kBlock * 128), tm, full, dh * 64, y[pg]);
          if (is_k)
            ++armed_k;
          else
            ++armed_v;
          return true;
        };
        // K runs three steps ahead of V: the scores of step j+3 are issued right after P V of j
        for (int j = max(pre_k, 0); j < min(kSBufs, nsteps) && ok; ++j) ok = load_kv(sel, cnt, h, G, j, true);
        if (pre_k > 0) armed_k = pre_k;
        pre_k = -1;
#pragma unroll 1
        for (int j = 0; j < nsteps && ok; ++j) {
          ok = load_kv(sel, cnt, h, Gv, j, false);
          if (ok && j + kSBufs < nsteps) ok = load_kv(sel, cnt, h, G, j + kSBufs, true);
        }
        if (ok && p.do_linear) {
          // hi and lo halves of the D x D state ride the V ring as two more "steps"
          for (int hl = 0; hl < 2 && ok; ++hl) {
            const int gj = Gv + nsteps + hl;
            const int s = gj % kStages;
            const uint32_t ph = (gj / kStages) & 1;
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
        // the Q tile has landed before the item ends (a tile without any step never looks at it)
        if (ok) ok = wait_bar(&bars->q_full, ic & 1, bars, p.status);
        if (!SPLIT && ok && item + item_stride < n_items) {
          // Next item: once this one's scores are all consumed (and phi(Q) is taken), the Q tile and
          // the K ring are free, so its Q and first K steps are requested under the epilogue.
          ok = wait_bar(&bars->final_known, ic & 1, bars, p.status);
          if (ok && p.do_linear) ok = wait_bar(&bars->lin_a_full, ic & 1, bars, p.status);
          if (ok && bars->final) {
            const Item N = get_item(item + item_stride);
            load_q(N.h, N.row0);
            pre_k = 0;
            for (int j = 0; j < min(kSBufs, N.nsteps) && ok; ++j) {
              ok = load_kv(N.sel, N.cnt, N.h, G + nsteps, j, true);
              if (ok) ++pre_k;
            }
          }
        }
        if (!ok) {
          // drain: let every copy already issued land before the CTA's shared memory goes away
          mbar_wait(&bars->q_full, ic & 1, 1u << 16);
          for (int i = 0; i < 2; ++i) {
            const int arms = i == 0 ? armed_k : armed_v;
            for (int a = max(0, arms - kStages); a < arms; ++a) {  // the last loads of each stage
              const int gj = (i == 0 ? G : Gv) + a;
              mbar_wait(i == 0 ? &bars->k_full[gj % kStages] : &bars->v_full[gj % kStages], (gj / kStages) & 1, 1u << 16);
            }
          }
          if (pre_k >= 0) {  // requests made for the next item
            mbar_wait(&bars->q_full, (ic + 1) & 1, 1u << 16);
            for (int a = 0; a < pre_k; ++a) {
              const int gj = G + nsteps + a;
              mbar_wait(&bars->k_full[gj % kStages], (gj / kStages) & 1, 1u << 16);
            }
          }
        }
      }
    } else if (warp == 1) {
      // ================================================================= MMA issuer
      if (leader) {
        constexpr uint32_t kHiSw = desc_hi_sw128(1024);
        const uint32_t q_lo = desc_lo_sw128(smem_u32(smem + L::kQ), 16);
        bool ok = true;
        if (!pre_qk) {
          ok = wait_bar(&bars->q_full, ic & 1, bars, p.status);
          tc_fence_after();
        }
        HSA_T(3011);
        // scores of step j of an item with xcnt pages whose steps start at gbase
        auto issue_qk = [&](int xcnt, int gbase, int j) -> bool {
          const int gj = gbase + j;
          const int s = gj % kStages;
          if (!wait_bar(&bars->k_full[s], (gj / kStages) & 1, bars, p.status)) return false;
          tc_fence_after();
          const uint32_t k_lo = desc_lo_sw128(smem_u32(smem + L::kK + s * L::kTile), 16);
          const uint32_t d_tmem = tmem + kColS + 128 * (gj % kSBufs);
          if (xcnt - 2 * j >= 2) {
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
          tc_commit(&bars->s_full[gj % kSBufs]);
          return true;
        };
        if (!pre_qk)
          for (int j = 0; j < min(kSBufs, nsteps) && ok; ++j) ok = issue_qk(cnt, G, j);
        pre_qk = false;
#pragma unroll 1
        for (int j = 0; j < nsteps && ok; ++j) {
          const int s = (Gv + j) % kStages;
          const int b = (G + j) % kSBufs;
          HSA_T(2048 + j * 8 + 0);
          ok = wait_bar(&bars->p_full[b], ((G + j) / kSBufs) & 1, bars, p.status);
          if (!ok) break;
          HSA_T(2048 + j * 8 + 1);
          ok = wait_bar(&bars->v_full[s], ((Gv + j) / kStages) & 1, bars, p.status);
          if (!ok) break;
          tc_fence_after();
          HSA_T(2048 + j * 8 + 2);
          constexpr uint32_t idesc = idesc_bf16_f32(128, D, 0, 1);
          const uint32_t v_lo = desc_lo_sw128(smem_u32(smem + L::kV + s * L::kTile), L::kHalf);
          const uint32_t o_acc = tmem + kColO;
          const uint32_t p_op = tmem + kColS + 128 * b;
          const uint32_t acc0 = j > 0 ? 1u : 0u;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            tc_mma_ts_lo(o_acc, p_op + kk * 8, v_lo + kk * 128, kHiSw, idesc, kk > 0 ? 1u : acc0);
          if (cnt - 2 * j >= 2) {
#pragma unroll
            for (int kk = 4; kk < 8; ++kk)
              tc_mma_ts_lo(o_acc, p_op + kk * 8, v_lo + kk * 128, kHiSw, idesc, 1u);
          }
          tc_commit(&bars->v_empty[s]);
          tc_commit(&bars->pv_done);
          HSA_T(2048 + j * 8 + 3);
          // the scores of step j+3 overwrite the P just consumed: issued after the P V above,
          // the tensor pipe runs them in order
          if (j + kSBufs < nsteps) ok = issue_qk(cnt, G, j + kSBufs);
          HSA_T(2048 + j * 8 + 4);
        }
        if (ok) {
          tc_commit(&bars->o_done);
          // every P of the item has been seen, so every step has had its say on the safe pass
          bars->final = (safe || bars->redo == 0) ? 1 : 0;
          mbar_arrive(&bars->final_known);
        }
        if (ok && p.do_linear) {
          ok = wait_bar(&bars->lin_a_full, ic & 1, bars, p.status);
          for (int hl = 0; hl < 2 && ok; ++hl) {
            const int gj = Gv + nsteps + hl;
            const int s = gj % kStages;
            ok = wait_bar(&bars->v_full[s], (gj / kStages) & 1, bars, p.status);
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
        if (!SPLIT && ok && item + item_stride < n_items && bars->final) {
          // Next item: its first scores are issued as soon as the groups have read this item's
          // accumulators out of TMEM (the linear branch borrows two score buffers), so that they
          // are ready when the groups come out of the epilogue.
          ok = wait_bar(&bars->o_free, ic & 1, bars, p.status);
          if (ok) ok = wait_bar(&bars->q_full, (ic + 1) & 1, bars, p.status);
          tc_fence_after();
          const Item N = get_item(item + item_stride);
          for (int j = 0; j < min(kSBufs, N.nsteps) && ok; ++j) ok = issue_qk(N.cnt, G + nsteps, j);
          pre_qk = ok;
        }
      }
    }
      if (!end_of_attempt()) break;
      safe = true;
      G = Gv = ic = 0;  // the barriers were initialised again
    }
    G += nsteps;
    Gv += nsteps + (p.do_linear ? 2 : 0);
    ++ic;
    if (bars->abort_flag) break;
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(HSA_SMREGS));
    int mc = 0;  // exponent references published so far (one per item that ran a fast pass with steps)
#pragma unroll 1
    for (int item = item0; item < n_items; item += item_stride) {
    const Item I = get_item(item);
    const int tile = I.tile, h = I.h, row0 = I.row0, cnt = I.cnt, nsteps = I.nsteps, nsplit = I.nsplit;
    const int32_t* sel = I.sel;
    const int slot = (tile * p.H + h) * nparts + part;  // this CTA's partial-result slot
    safe = false;
#pragma unroll 1
    for (int attempt = 0; attempt < 2; ++attempt) {
      // ================================================================= softmax groups + epilogue
      const int grp = (warp - 4) >> 2;  // group g takes the steps j = g (mod 3)
      const int quad = warp & 3;        // TMEM lane quadrant this warp may access
      const int r = quad * 32 + lane;   // row inside the tile
      const int row = row0 + r;         // query index inside the chunk
      const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
      const uint32_t o_tmem = tmem + lane_off + kColO;
      const int64_t qpos = p.q_pos0 + row;
      const int64_t vis_end = p.causal ? min64(p.n_tokens, qpos + 1) : p.n_tokens;
      // the first row of the tile sees the fewest keys: a step whose pages all end at or before
      // that row's limit needs no masking
      const int64_t tile_vis_end = p.causal ? min64(p.n_tokens, p.q_pos0 + row0 + 1) : p.n_tokens;
      const float sl2 = p.scale_log2;
      // fast pass: t_ref is the fixed exponent reference (log2 domain) of the row;
      // safe pass: m_used is the running reference maximum (raw score units) with lazy rescale
      float t_ref = 0.f;
      float m_used = -INFINITY;
      float l = 0.f;
      bool ok = true;
      const int first = safe ? (grp == 0 ? 0 : nsteps) : grp;
      const int stride = safe ? 1 : kGroups;

      // ---- linear branch operands, prepared before the loop
      constexpr int HC = D / 2;
      const bool epi = grp < 2;
      const int cbase = (grp & 1) * HC;
      if (quad == 0) HSA_T(3014 + grp);
      // block ids of the next step are fetched one step ahead, off the critical path
      int nb0 = 0, nb1 = 0;
      if (first < nsteps) {
        nb0 = sel[2 * first];
        nb1 = (2 * first + 1 < cnt) ? sel[2 * first + 1] : 0;
      }
      // fast pass: the two groups alternate on the exponential phase.  Both are bound by the same
      // SFU pipe there, so running the phases one after the other costs nothing and lets each
      // group's loads, stores and barrier traffic hide under the other's exponentials.
      if (kTokens && !safe && grp == 1) mbar_arrive(&bars->tok[0]);
      int tok_i = 0;
#pragma unroll 1
      for (int j = first; j < nsteps; j += stride) {
        int blk0 = nb0, blk1 = nb1;
        if (j + stride < nsteps) {
          nb0 = sel[2 * (j + stride)];
          nb1 = (2 * (j + stride) + 1 < cnt) ? sel[2 * (j + stride) + 1] : 0;
        }
        const int b = (G + j) % kSBufs;
        const uint32_t s_tmem = tmem + lane_off + kColS + 128 * b;
        if (quad == 0) HSA_T(grp * 1024 + (j / kGroups) * 8 + 0);
        ok = __all_sync(0xffffffffu, wait_bar(&bars->s_full[b], ((G + j) / kSBufs) & 1, bars, p.status));
        if (!ok) break;
        tc_fence_after();
        if (quad == 0) HSA_T(grp * 1024 + (j / kGroups) * 8 + 1);
        uint32_t cbuf[2][32];  // two 32-column chunks of the score row in flight
        // the first chunk is requested at once: its latency runs under the bookkeeping below
        // (the steps that look for the row maximum first issue their own loads)
        const bool early_ld = !(safe || j == 0);
        if (early_ld) tmem_ld32(s_tmem, cbuf[0]);
        const int npg = min(2, cnt - 2 * j);
        const int n = npg * kBlock;
        if (blk0 < 0 || blk0 >= p.n_blocks) blk0 = 0;
        if (blk1 < 0 || blk1 >= p.n_blocks) blk1 = 0;
        const int64_t last_blk = blk0 > blk1 ? blk0 : blk1;
        const bool need_mask = (n != 128) || (last_blk * kBlock + kBlock > tile_vis_end);
        // visible keys per page: columns [0, lim) of the page's 64
        int lim0 = kBlock, lim1 = kBlock;
        if (need_mask) {
          lim0 = static_cast<int>(max64(0, min64(kBlock, vis_end - static_cast<int64_t>(blk0) * kBlock)));
          lim1 = npg > 1 ? static_cast<int>(max64(0, min64(kBlock, vis_end - static_cast<int64_t>(blk1) * kBlock))) : 0;
        }
        const int nchunks = n / 32;
        if (safe || j == 0) {
          // the reference needs the row maximum first: a pass over the score row in chunks
          float mxa = -INFINITY, mxb = -INFINITY;
          tmem_ld32(s_tmem, cbuf[0]);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            if (c < nchunks) {
              tc_wait_ld();
              if (c + 1 < nchunks) tmem_ld32(s_tmem + 32 * (c + 1), cbuf[(c + 1) & 1]);
              uint32_t(&x)[32] = cbuf[c & 1];
              if (need_mask) {
                const int lim = ((c >> 1) ? lim1 : lim0) - (c & 1) * 32;
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (i >= lim) x[i] = 0xff800000u;  // -inf
              }
#pragma unroll
              for (int i = 0; i < 32; i += 4) {
                mxa = fmax3(mxa, __uint_as_float(x[i]), __uint_as_float(x[i + 1]));
                mxb = fmax3(mxb, __uint_as_float(x[i + 2]), __uint_as_float(x[i + 3]));
              }
            }
          }
          const float m_new = fmaxf(mxa, mxb);
          if (!safe) {
            // fix the row's reference for the whole tile and hand it to the other group
            t_ref = (m_new == -INFINITY) ? 0.f : fmaf(m_new, sl2, kHeadroom);
            bars->mref[r] = t_ref;
            mbar_arrive(&bars->mref_ready);
          } else {
            // lazy rescale: move the reference only when it would grow by more than 2^8
            float factor = 1.f;
            if (m_used == -INFINITY) {
              m_used = m_new;  // nothing accumulated so far
            } else if ((m_new - m_used) * sl2 > 8.f) {
              factor = ex2((m_used - m_new) * sl2);
              l *= factor;
              m_used = m_new;
            }
            if (j > 0) {
              // O must be quiescent: the previous P V has to be complete before it is rescaled
              ok = __all_sync(0xffffffffu, wait_bar(&bars->pv_done, (G + j - 1) & 1, bars, p.status));
              if (!ok) break;
              tc_fence_after();
              if (__any_sync(0xffffffffu, factor != 1.f)) {
#pragma unroll 1
                for (int c0 = 0; c0 < D; c0 += 32) {
                  uint32_t o[32];
                  tmem_ld32(o_tmem + c0, o);
                  tc_wait_ld();
#pragma unroll
                  for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
                  tmem_st32(o_tmem + c0, o);
                }
                tc_wait_st();
              }
            }
            t_ref = (m_used == -INFINITY) ? 0.f : m_used * sl2;
          }
        } else if (j < kGroups) {
          // first step of groups 1 and 2 in the fast pass: take the reference group 0 fixed
          ok = __all_sync(0xffffffffu, wait_bar(&bars->mref_ready, mc & 1, bars, p.status));
          if (!ok) break;
          t_ref = bars->mref[r];
        }
        if (quad == 0) HSA_T(grp * 1024 + (j / kGroups) * 8 + 2);
        // exponentials in four chunks of 32 columns: the load of the next chunk and the store of
        // the previous P chunk run under the arithmetic of the current one
        const float nt = -t_ref;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};  // independent partial row sums
        if (!early_ld) tmem_ld32(s_tmem, cbuf[0]);
        if (kTokens && !safe) {
          ok = __all_sync(0xffffffffu, wait_bar(&bars->tok[grp], tok_i & 1, bars, p.status));
          if (!ok) break;
          ++tok_i;
        }
        if (quad == 0) HSA_T(grp * 1024 + (j / kGroups) * 8 + 3);
#if HSA_CONTINUOUS
        if (nchunks == 4 && !need_mask) {
          // full, unmasked step (the usual case): ONE software pipeline over the 128 columns --
          // scale-and-shift of column i, exponential of column i - LAG, row sum and bf16 pack of
          // column i - 2 LAG -- that does not drain at the chunk boundaries; the TMEM load of the next
          // chunk is issued when the pipeline enters a chunk, the P store when it leaves one
          constexpr int LAG = HSA_CONTINUOUS;
          float y[128];
          uint32_t pk[2][16];
#pragma unroll
          for (int i = 0; i < 128 + 2 * LAG; ++i) {
            if (i < 128) {
              if ((i & 31) == 0) {
                tc_wait_ld();
                if (i + 32 < 128) tmem_ld32(s_tmem + i + 32, cbuf[((i >> 5) + 1) & 1]);
              }
              y[i] = fmaf(__uint_as_float(cbuf[(i >> 5) & 1][i & 31]), sl2, nt);
            }
            if (i >= LAG && i - LAG < 128) y[i - LAG] = ex2v(y[i - LAG]);
            if (i >= 2 * LAG && i - 2 * LAG < 128) {
              const int k = i - 2 * LAG;
              acc[k & 3] += y[k];
              if (k & 1) pk[(k >> 5) & 1][(k & 31) >> 1] = pack_bf16(y[k - 1], y[k]);
              if ((k & 31) == 31) tmem_st16(s_tmem + 16 * (k >> 5), pk[(k >> 5) & 1]);
            }
          }
        } else
#endif
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          if (c < nchunks) {
            tc_wait_ld();
            if (c + 1 < nchunks) tmem_ld32(s_tmem + 32 * (c + 1), cbuf[(c + 1) & 1]);
            uint32_t(&x)[32] = cbuf[c & 1];
            if (need_mask) {
              const int lim = ((c >> 1) ? lim1 : lim0) - (c & 1) * 32;  // visible columns of this chunk
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (i >= lim) x[i] = 0xff800000u;  // -inf
            }
#if HSA_INTERLEAVE
            // software pipeline over the chunk's 32 columns: scale-and-shift of column i, the
            // exponential of column i - LAG and the row sum / bf16 pack of column i - LAG - LAG2 are
            // issued next to each other, so that the FMA-pipe work fills the issue slots between
            // two exponentials (the SFU takes one warp instruction per 8 cycles)
            float y[32];
            uint32_t pk[16];
            constexpr int LAG = HSA_INTERLEAVE;
            constexpr int LAG2 = LAG;
#pragma unroll
            for (int i = 0; i < 32 + LAG + LAG2; ++i) {
              if (i < 32) y[i] = fmaf(__uint_as_float(x[i]), sl2, nt);
              if (i >= LAG && i - LAG < 32) y[i - LAG] = ex2v(y[i - LAG]);
              if (i >= LAG + LAG2 && i - LAG - LAG2 < 32) {
                const int k = i - LAG - LAG2;
                acc[k & 3] += y[k];
                if (k & 1) pk[k >> 1] = pack_bf16(y[k - 1], y[k]);
              }
            }
#else
            // stage by stage over the whole chunk, so that 32 independent operations of each kind
            // are in flight: scale-and-shift, exponential, row sum, bf16 pack
            float y[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) y[i] = fmaf(__uint_as_float(x[i]), sl2, nt);
#pragma unroll
            for (int i = 0; i < 32; ++i) y[i] = ex2(y[i]);
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              acc[0] += y[i];
              acc[1] += y[i + 1];
              acc[2] += y[i + 2];
              acc[3] += y[i + 3];
            }
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 32; i += 2) pk[i >> 1] = pack_bf16(y[i], y[i + 1]);
#endif
            tmem_st16(s_tmem + 16 * c, pk);
            if (quad == 0) HSA_T(3100 + grp * 256 + (j / kGroups) * 8 + c);
          }
        }
        {
          const float lstep = (acc[0] + acc[1]) + (acc[2] + acc[3]);
          l += lstep;
          // a weight far above the fixed reference: finite here, but the tile is redone safely
          if (!safe && !(lstep <= kRedoSum)) bars->redo = 1;
        }
        if (kTokens && !safe) mbar_arrive(&bars->tok[grp ^ 1]);
        if (quad == 0) HSA_T(grp * 1024 + (j / kGroups) * 8 + 4);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(&bars->p_full[b]);
        if (quad == 0) HSA_T(grp * 1024 + (j / kGroups) * 8 + 5);
      }

      // ---- linear branch operands (Q is still in shared memory: the next item's tile is requested only
      //      after phi(Q) has been handed over)
      float den_part = 0.f, den_part2 = 0.f;
      uint32_t fr[HC / 2];
      if (ok && p.do_linear && epi) {
        // phi(q) of this thread's row for its half of the dims (bf16 A operand of the linear
        // MMA) and the partial denominator phi(q) . z -- after the group's last step, while the
        // tensor pipe finishes the item's last products
        ok = __all_sync(0xffffffffu, wait_bar(&bars->q_full, ic & 1, bars, p.status));
        if (quad == 0) HSA_T(3012 + grp);
        const uint8_t* qrow = smem + L::kQ + r * 128;
        const float4* z4 = reinterpret_cast<const float4*>(p.z + static_cast<size_t>(h) * D + cbase);
#pragma unroll
        for (int c16 = 0; c16 < HC / 8; ++c16) {
          const float4 za = z4[c16 * 2], zb = z4[c16 * 2 + 1];
          const float z[8] = {za.x, za.y, za.z, za.w, zb.x, zb.y, zb.z, zb.w};
          const int cc = cbase / 8 + c16;  // 16-byte chunk of the row
          const int dh = cc >> 3, ch = cc & 7;
          const uint4 raw = *reinterpret_cast<const uint4*>(qrow + dh * L::kHalf + ((ch ^ (r & 7)) << 4));
          const uint32_t* qw = reinterpret_cast<const uint32_t*>(&raw);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint32_t pk = pack_bf16(phi_elu1(__uint_as_float(qw[i] << 16)), phi_elu1(__uint_as_float(qw[i] & 0xffff0000u)));
            fr[c16 * 4 + i] = pk;
            // the denominator uses the rounded values the MMA will see
            den_part = fmaf(__uint_as_float(pk << 16), z[2 * i], den_part);
            den_part2 = fmaf(__uint_as_float(pk & 0xffff0000u), z[2 * i + 1], den_part2);
          }
        }
        den_part += den_part2;
      }

      // ---------------------------------------------------------------- epilogue
      // (this group's columns of the output row: group 0 -> [0, D/2), group 1 -> [D/2, D))
      if (ok && nsteps > 0) {
        ok = __all_sync(0xffffffffu, wait_bar(&bars->o_done, ic & 1, bars, p.status));
        tc_fence_after();
      }
      if (quad == 0) HSA_T(3002 + grp);
      if (ok && p.do_linear && epi) {
        if constexpr (D == 128) {
          tmem_st32(tmem + lane_off + kColPhi + grp * 32, reinterpret_cast<uint32_t(&)[32]>(fr[0]));
        } else {
          tmem_st16(tmem + lane_off + kColPhi + grp * 16, reinterpret_cast<uint32_t(&)[16]>(fr[0]));
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(&bars->lin_a_full);
      }
      // publish this group's partial row sum and denominator, then read the other group's
      bars->stat[grp][r] = make_float2(l, den_part);
      if (quad == 0) HSA_T(3004 + grp);
      named_bar_sync(1, 128 * kGroups);
      float lsum = 0.f, den = 0.f;
#pragma unroll
      for (int gg = 0; gg < kGroups; ++gg) {
        const float2 st = bars->stat[gg][r];
        lsum += st.x;
        den += st.y;
      }
      float inv_l = (nsteps > 0 && lsum > 0.f) ? 1.f / lsum : 0.f;
      const bool has_o = nsteps > 0;
      // Split tile: every part dumps its unnormalised accumulator with the row sums and the
      // exponent references, then takes a ticket; the part that draws the last ticket merges all of
      // them (its own included) in the epilogue below, the others write no output.  Only the attempt
      // that stands (no redo pending) takes part.
      const bool final_attempt = safe || bars->redo == 0;
      bool do_output = final_attempt;
      float pf[SPLIT ? kFwdSplitMax : 1];  // merge factors 2^(ref_p - max ref) of the parts (split tiles only)
      if (SPLIT && nsplit > 1 && final_attempt) {
        if (ok) {
          float* po = p.part_o + (static_cast<size_t>(slot) * kTileM + r) * D + cbase;
#pragma unroll 1
          for (int c0 = 0; c0 < HC; c0 += 16) {
            uint32_t oa[16];
            tmem_ld16(o_tmem + cbase + c0, oa);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; i += 4)
              *reinterpret_cast<float4*>(po + c0 + i) =
                  make_float4(__uint_as_float(oa[i]), __uint_as_float(oa[i + 1]), __uint_as_float(oa[i + 2]),
                              __uint_as_float(oa[i + 3]));
          }
          if (grp == 0) {
            p.part_l[static_cast<size_t>(slot) * kTileM + r] = lsum;
            p.part_ref[static_cast<size_t>(slot) * kTileM + r] = t_ref;
          }
          __threadfence();
        }
        named_bar_sync(3, 128 * kGroups);
        if (warp == 4 && lane == 0) {
          int32_t* tk = p.part_ticket + tile * p.H + h;
          const int t = ok ? atomicAdd(tk, 1) : -1;
          if (t == nsplit - 1) *tk = 0;  // the counter is back at zero for the next launch
          bars->ticket = t;
        }
        named_bar_sync(3, 128 * kGroups);
        do_output = bars->ticket == nsplit - 1;
        if (do_output) {
          __threadfence();
          // common reference R = largest reference among the parts that saw a key for this row
          const size_t s0 = static_cast<size_t>(slot - part) * kTileM + r;
          float rmax = -INFINITY;
          for (int q = 0; q < nsplit; ++q)
            if (__ldcg(&p.part_l[s0 + static_cast<size_t>(q) * kTileM]) > 0.f)
              rmax = fmaxf(rmax, __ldcg(&p.part_ref[s0 + static_cast<size_t>(q) * kTileM]));
          float ltot = 0.f;
#pragma unroll
          for (int q = 0; q < (SPLIT ? kFwdSplitMax : 1); ++q) {
            pf[q] = 0.f;
            if (q < nsplit) {
              const float lq = __ldcg(&p.part_l[s0 + static_cast<size_t>(q) * kTileM]);
              if (lq > 0.f) {
                pf[q] = ex2(__ldcg(&p.part_ref[s0 + static_cast<size_t>(q) * kTileM]) - rmax);
                ltot = fmaf(lq, pf[q], ltot);
              }
            }
          }
          inv_l = ltot > 0.f ? 1.f / ltot : 0.f;
        }
      }
      // the linear numerator is final once the MMA lane's commit has arrived
      auto wait_lin = [&]() {
        if (ok && p.do_linear && epi) {
          ok = __all_sync(0xffffffffu, wait_bar(&bars->lin_done, ic & 1, bars, p.status));
          tc_fence_after();
        }
      };
      if (!(epi && do_output)) wait_lin();
      if (quad == 0) HSA_T(3006 + grp);
      // The output tile is staged in the V stage that held the last step's values (the state
      // halves, if any, sit in the other two): free since the last P V, and not loaded again before
      // the next item, which starts after the store below has read it.
      uint8_t* stage_out = smem + L::kV + ((Gv + nsteps + 2) % kStages) * L::kTile;
      if (ok && epi && do_output) {  // warp-uniform: the TMEM loads below are warp-collective
        const bool wr = row < p.n_q;  // rows past the end of the chunk compute but never store
        float lin_den = den;
        const float* lnum = nullptr;
        if (wr && p.do_linear && p.lin_num != nullptr) {
          lnum = p.lin_num + (static_cast<size_t>(row) * p.H + h) * D;
          lin_den += p.lin_den[static_cast<size_t>(row) * p.H + h];
        }
        const float inv_den = (p.do_linear && lin_den > 0.f) ? 1.f / lin_den : 0.f;
        const __nv_bfloat16* gl =
            (wr && p.g_lin) ? p.g_lin + static_cast<size_t>(row) * p.g_ts + static_cast<size_t>(h) * p.g_hs : nullptr;
        const __nv_bfloat16* gs =
            (wr && p.g_sp) ? p.g_sp + static_cast<size_t>(row) * p.g_ts + static_cast<size_t>(h) * p.g_hs : nullptr;
        const __nv_bfloat16* ext =
            (wr && p.ext_lin) ? p.ext_lin + (static_cast<size_t>(row) * p.H + h) * D : nullptr;
        const int g_ds = static_cast<int>(p.g_ds);
        const bool sig = p.gate_act == 1;
        // (decided from the launch parameters, not from this thread's pointers: the branch holds
        // warp-collective TMEM loads and must not diverge inside a warp)
        const bool plain = !p.g_lin && !p.g_sp && !(p.do_linear && p.lin_num != nullptr) && !p.ext_lin &&
                           !(SPLIT && nsplit > 1);
        if (plain) {
          // no gates, no causal partials, no external linear output, no merge.  The sparse part is
          // read and scaled first, while the tensor pipe still works on the linear numerator.
          const float il = has_o ? inv_l : 0.f, id = p.do_linear ? inv_den : 0.f;
          float osp[HC];
#pragma unroll
          for (int c0 = 0; c0 < HC; c0 += 32) {
            uint32_t oa[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) oa[i] = 0u;
            if (has_o) {
              tmem_ld32(o_tmem + cbase + c0, oa);
              tc_wait_ld();
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) osp[c0 + i] = __uint_as_float(oa[i]) * il;
          }
          wait_lin();
#pragma unroll
          for (int c0 = 0; c0 < HC; c0 += 32) {
            uint32_t ln[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) ln[i] = 0u;
            if (p.do_linear) {
              tmem_ld32(tmem + lane_off + kColLin + cbase + c0, ln);
              tc_wait_ld();
            }
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 32; i += 2)
              pk[i >> 1] = pack_bf16(fmaf(__uint_as_float(ln[i]), id, osp[c0 + i]),
                                     fmaf(__uint_as_float(ln[i + 1]), id, osp[c0 + i + 1]));
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              const int cc = ((cbase + c0) >> 3) + q4;  // 16-byte chunk of the row
              *reinterpret_cast<uint4*>(stage_out + (cc >> 3) * L::kHalf + r * 128 + (((cc & 7) ^ (r & 7)) << 4)) =
                  make_uint4(pk[4 * q4], pk[4 * q4 + 1], pk[4 * q4 + 2], pk[4 * q4 + 3]);
            }
          }
        } else {
          wait_lin();
        }
        // rolled on purpose: 16 columns per trip keeps this once-per-tile code small
#pragma unroll 1
        for (int c0 = cbase; c0 < (plain ? cbase : cbase + HC); c0 += 16) {
          uint32_t oa[16], ln[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) oa[i] = ln[i] = 0u;
          if (quad == 0) HSA_T(3040 + grp * 16 + ((c0 - cbase) / 16) * 3 + 0);
          if (SPLIT && nsplit > 1) {
            // merged accumulator: sum over the parts of factor * partial, from the dumps
            float acc[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] = 0.f;
            const float* po = p.part_o + (static_cast<size_t>(slot - part) * kTileM + r) * D + c0;
#pragma unroll
            for (int q = 0; q < (SPLIT ? kFwdSplitMax : 1); ++q) {
              if (q < nsplit && pf[q] != 0.f) {
#pragma unroll
                for (int i = 0; i < 16; i += 4) {
                  const float4 v = __ldcg(reinterpret_cast<const float4*>(po + static_cast<size_t>(q) * kTileM * D + i));
                  acc[i] = fmaf(pf[q], v.x, acc[i]);
                  acc[i + 1] = fmaf(pf[q], v.y, acc[i + 1]);
                  acc[i + 2] = fmaf(pf[q], v.z, acc[i + 2]);
                  acc[i + 3] = fmaf(pf[q], v.w, acc[i + 3]);
                }
              }
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) oa[i] = __float_as_uint(acc[i]);
          } else if (has_o) {
            tmem_ld16(o_tmem + c0, oa);
          }
          if (p.do_linear) tmem_ld16(tmem + lane_off + kColLin + c0, ln);
          tc_wait_ld();
          if (quad == 0) HSA_T(3040 + grp * 16 + ((c0 - cbase) / 16) * 3 + 1);
          uint32_t packed[8];
          {
          // gate weights and causal partials are fetched under ONE branch each per trip (a branch
          // per element costs far more than the arithmetic it guards)
          float wl[16], ws[16], ladd[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            wl[i] = 1.f;
            ws[i] = 1.f;
            ladd[i] = 0.f;
          }
          if (gl) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float w0 = __bfloat162float(gl[(c0 + i) * g_ds]);
              wl[i] = sig ? __fdividef(1.f, 1.f + __expf(-w0)) : w0;
            }
          }
          if (gs) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float w0 = __bfloat162float(gs[(c0 + i) * g_ds]);
              ws[i] = sig ? __fdividef(1.f, 1.f + __expf(-w0)) : w0;
            }
          }
          if (lnum) {
#pragma unroll
            for (int i = 0; i < 16; ++i) ladd[i] = lnum[c0 + i];
          }
          if (ext) {  // linear branch computed by an earlier pass (Linformer form): already normalised
            const uint4 e0 = *reinterpret_cast<const uint4*>(ext + c0);
            const uint4 e1 = *reinterpret_cast<const uint4*>(ext + c0 + 8);
            const __nv_bfloat162* b0 = reinterpret_cast<const __nv_bfloat162*>(&e0);
            const __nv_bfloat162* b1 = reinterpret_cast<const __nv_bfloat162*>(&e1);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 f0 = __bfloat1622float2(b0[i]), f1 = __bfloat1622float2(b1[i]);
              ladd[2 * i] = f0.x;
              ladd[2 * i + 1] = f0.y;
              ladd[8 + 2 * i] = f1.x;
              ladd[8 + 2 * i + 1] = f1.y;
            }
          }
#pragma unroll
          for (int i = 0; i < 16; i += 2) {
            float res[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const float osp = has_o ? __uint_as_float(oa[i + e]) * inv_l : 0.f;
              const float olin = p.do_linear ? (__uint_as_float(ln[i + e]) + ladd[i + e]) * inv_den
                                             : ladd[i + e];  // 0 unless an external linear output is given
              res[e] = fmaf(wl[i + e], olin, ws[i + e] * osp);
            }
            packed[i >> 1] = pack_bf16(res[0], res[1]);
          }
          }
          if (quad == 0) HSA_T(3040 + grp * 16 + ((c0 - cbase) / 16) * 3 + 2);
          // stage the row (each thread touches only its own) in the 128-byte-swizzled layout the
          // output tensor map expects
          {
            const int cc = c0 >> 3;  // 16-byte chunk of the row
            uint8_t* srow = stage_out + (cc >> 3) * L::kHalf + r * 128;
            *reinterpret_cast<uint4*>(srow + (((cc & 7) ^ (r & 7)) << 4)) =
                make_uint4(packed[0], packed[1], packed[2], packed[3]);
            *reinterpret_cast<uint4*>(srow + ((((cc + 1) & 7) ^ (r & 7)) << 4)) =
                make_uint4(packed[4], packed[5], packed[6], packed[7]);
          }
        }
      }
      // the accumulators of this item have been read: the tensor pipe may start on the next item
      tc_fence_before();
      mbar_arrive(&bars->o_free);
      // both epilogue groups have staged their columns: one elected thread stores the tile
      // (rows past the end of the chunk are clipped by the tensor map)
      fence_proxy_async_smem();
      named_bar_sync(2, 128 * kGroups);
      if (ok && do_output && warp == 4) {
        if (elect_one_sync()) {
          for (int dh = 0; dh < DH; ++dh) tma_store_3d(&tm_out, stage_out + dh * L::kHalf, dh * 64, h, row0);
          tma_store_commit();
          tma_store_wait_read();  // the tile must stay in shared memory until it has been read
        }
      }
      if (quad == 0) HSA_T(3008 + grp);
      if (!end_of_attempt()) break;
      safe = true;
      G = Gv = ic = mc = 0;  // the barriers were initialised again
    }
    if (nsteps > 0 && !safe) ++mc;  // group 0 published a reference in the fast pass
    G += nsteps;
    Gv += nsteps + (p.do_linear ? 2 : 0);
    ++ic;
    if (bars->abort_flag) break;
    }
  }

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

static int g_fwd_sms = 0;  // SMs of the device: the persistent kernel runs one CTA on each

cudaError_t forward_init() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&g_fwd_sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(hsa_forward_kernel<128, false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<128>::kTotal);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(hsa_forward_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Smem<128>::kTotal);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(hsa_forward_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Smem<64>::kTotal);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(hsa_forward_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Smem<64>::kTotal);
  return e;
}

cudaError_t launch_forward(const FwdParams& p, int D, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                           const CUtensorMap& tm_v, const CUtensorMap& tm_state, const CUtensorMap& tm_out,
                           cudaStream_t st) {
  const int n_tiles = (p.n_q + kTileM - 1) / kTileM;
  const bool split = p.max_splits > 1;
  // split: one CTA per (tile, head, part); plain: one persistent CTA per SM over the (tile, head) items
  const int n_items = n_tiles * p.H;
  dim3 grid(n_tiles, p.H, p.max_splits);
  if (!split) grid = dim3(n_items < g_fwd_sms ? n_items : (g_fwd_sms > 0 ? g_fwd_sms : 1), 1, 1);
  if (D == 128) {
    if (split)
      hsa_forward_kernel<128, true><<<grid, kThreads, Smem<128>::kTotal, st>>>(tm_q, tm_k, tm_v, tm_state, tm_out, p);
    else
      hsa_forward_kernel<128, false><<<grid, kThreads, Smem<128>::kTotal, st>>>(tm_q, tm_k, tm_v, tm_state, tm_out, p);
  } else {
    if (split)
      hsa_forward_kernel<64, true><<<grid, kThreads, Smem<64>::kTotal, st>>>(tm_q, tm_k, tm_v, tm_state, tm_out, p);
    else
      hsa_forward_kernel<64, false><<<grid, kThreads, Smem<64>::kTotal, st>>>(tm_q, tm_k, tm_v, tm_state, tm_out, p);
  }
  return cudaGetLastError();
}

}  // namespace hsa
