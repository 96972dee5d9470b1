// hsa_forward kernel for sm_100a.
//
// One CTA per (128-row query tile, head), 384 threads in three warpgroups:
//   warp 0       TMA producer: Q tile, then the selected K/V pages gathered through the page
//                table (two 64-token pages = 128 keys per step) into two 3-stage rings, then the
//                hi/lo halves of the linear state; also owns the TMEM allocation
//   warp 1       tcgen05.mma issuer: S = Q K^T three steps ahead, O += P V with P read from
//                TMEM, then the linear numerator phi(Q) S
//   warp 2       (one lane, once) asks a slice of the group's block list into L2 ahead of the rings
//   warps 4..11  two softmax groups of four warps: group g takes the KV steps j = g (mod 2);
//                one query row per thread
// The kernel is launched as a programmatic dependent of the kernel before it (block selection)
// and waits for it on entry.
// TMEM: O (128 fp32 columns) | three S buffers (128 columns each); P overwrites the first 64
// columns of its S buffer as packed bf16.  With three score buffers the tensor pipe never waits
// for a softmax group: Q K^T of step j+3 is issued right after P V of step j.
//
// Both groups accumulate into ONE O.  That needs a common exponent reference per row, so in the
// normal ("fast") pass the reference is fixed once: the row maximum over the first 32 keys of the
// first step (all of its keys when the step is masked) plus a headroom of 2^20.  Every later weight is exp2(s - ref) with no running maximum and no rescale.
// fp32 / bf16 carry the same relative precision at any magnitude, so the result equals the
// usual online softmax as long as no weight overflows; a step whose weights exceed 2^27 sets a
// flag and the tile is redone in a "safe" pass: one group, classic online softmax with lazy
// rescale.  The two groups' partial row sums are added in the epilogue, which also applies the
// linear branch and the gates and stores bf16 once.
// Every barrier wait is bounded; when one gives up the kernel records a timeout in the status
// word and all roles drain to the common exit.
//
// LINF (the Linformer form of the linear branch, Sec. 3.3 Eq. 3): the loop has two segments.  The
// first runs over every page of the compressed pool (K~, V~), the second over the selected pages;
// each segment has its own accumulator in TMEM (O_lin | O_sp), its own exponent reference and its
// own row sums, and the epilogue merges the two normalised results.  TMEM then holds two score
// buffers instead of three: O_sp | O_lin | S0 | S1.
#include <cuda_bf16.h>

#include "hsa_internal.h"
#include "ptx.cuh"

namespace hsa {

namespace {

constexpr int kGroups = 2;     // softmax groups; group g takes the KV steps j = g (mod kGroups)
constexpr int kSoftmaxRegs = 224;  // registers per softmax thread after the hand-over (56 for the others)
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
  static constexpr int kStats = kK;  // float[2][128][4], reuses K stage 0 once the loop is over
  static constexpr int kBars = kTile + 2 * kStages * kTile;
  static constexpr int kTotal = kBars + 1536 + 1024;  // barriers + per-row references, + slack
};

struct Bars {
  uint64_t q_full;
  int ticket;  // split tiles: arrival number of this CTA among the parts of its (tile, head)
  uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  uint64_t s_full[kSBufs];
  uint64_t p_full[kSBufs];
  uint64_t pv_done;
  uint64_t o_done;
  uint64_t mref_ready[2];  // per loop segment
  uint64_t lin_a_full;
  uint64_t lin_done;
  uint32_t tmem_base;
  volatile int abort_flag;
  volatile int redo;
  float mref[2][128];  // per-row exponent reference (log2 domain) of the fast pass, per loop segment
};
static_assert(sizeof(Bars) <= 1536, "barrier block must fit its shared-memory slot");

constexpr int kExpLag = 8;  // columns between scale-and-shift, exponential and row sum in the softmax pipeline

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
// either feature map without a branch: max(x, 0) + w * exp(min(x, 0)) with w = 1 (elu + 1) or 0 (relu)
__device__ __forceinline__ float phi_q(float x, float w) {
  return fmaf(w, ex2(fminf(x, 0.f) * 1.4426950408889634f), fmaxf(x, 0.f));
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float m;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(m) : "f"(a), "f"(b), "f"(c));
  return m;
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
  for (int i = 0; i < 2; ++i) mbar_init(&bars->mref_ready[i], 128);  // one group publishes the per-row reference
  mbar_init(&bars->lin_a_full, 256);
  mbar_init(&bars->lin_done, 1);
  bars->redo = 0;
  fence_mbar_init();
}

}  // namespace

// SPLIT: compiled with the split-tile path (grid z > 1); the plain kernel carries none of it
// LINF: compiled with the compressed-pool segment in front of the selected pages (tm_kc, tm_vc)
template <int D, bool SPLIT, bool LINF>
__global__ void __launch_bounds__(kThreads, 1)
hsa_forward_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v,
                   const __grid_constant__ CUtensorMap tm_state,
                   const __grid_constant__ CUtensorMap tm_out, const __grid_constant__ CUtensorMap tm_kc,
                   const __grid_constant__ CUtensorMap tm_vc, const FwdParams p) {
  static_assert(!(SPLIT && LINF), "split lists and the compressed segment are not combined");
  constexpr int NSB = LINF ? 2 : kSBufs;                 // score buffers in use
  constexpr uint32_t kColSb = LINF ? 256 : kColS;        // first score buffer
  constexpr uint32_t kColLn = LINF ? 128 : kColLin;      // linear-branch accumulator
  using L = Smem<D>;
  constexpr int DH = D / 64;  // 64-element (128-byte) slabs per row
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  Bars* bars = reinterpret_cast<Bars*>(smem + L::kBars);
  float* stats = reinterpret_cast<float*>(smem + L::kStats);  // [group][row][l, den, -, -]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // barriers, TMEM allocation and the CTA-wide barrier that publishes them
  auto setup = [&]() {
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
  };
  // Launched with programmatic stream serialization: this grid may be scheduled while the kernel
  // before it (block selection) is still extracting its lists.  Nothing of that kernel's output is
  // read before the wait; the plain kernel does its set-up first, under that kernel's tail (a split
  // CTA may still leave without any set-up, so it sets up after it has seen its list).
  if (!SPLIT) setup();
  asm volatile("griddepcontrol.wait;" ::: "memory");
  int tile = blockIdx.x, h = blockIdx.y, part = blockIdx.z;
  // Parts of a list of `st` two-page steps.  balance > 0: the steps one SM would run if the whole
  // launch were spread evenly; a list is cut into the fewest parts none of which is longer than that
  // (no part shorter than 16 steps).  balance == 0: parts of split_blocks blocks.
  auto parts_of = [&](int st, int balance) -> int {
    const int want = balance > 0 ? min((st + balance - 1) / balance, max(1, st / 16))
                                 : (st + p.split_blocks / 2 - 1) / (p.split_blocks / 2);
    int ns = min(p.max_splits, max(1, want));
    const int per = (st + ns - 1) / ns;
    if (per > 0) ns = (st + per - 1) / per;  // no empty part
    return ns;
  };
  int balance = 0;
  if (SPLIT && p.remap) {
    // Longest lists first.  With one list per head every (tile, part) of a head costs the same, so the
    // heads are ranked by the steps one part of theirs takes and the grid walks through them in that
    // order (part-major inside a head: CTAs that run side by side gather the same pages); the heavy
    // parts start in the first wave and the short lists fill the tail.  Every warp works the mapping
    // out for itself from the H list lengths (a few dozen shuffles), so nothing has to be shared.
    const int n_tiles = p.n_tiles;
    int my_cnt = (lane < p.H && p.do_sparse) ? p.sel_cnt[lane] : 0;
    my_cnt = max(0, min(my_cnt, min(p.kcap, p.n_blocks)));
    const int st = (my_cnt + 1) / 2;
    int total = st;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    balance = max(1, static_cast<int>((static_cast<int64_t>(total) * n_tiles + p.nsm - 1) / p.nsm));
    const int ns = parts_of(st, balance);
    const int per = (st + ns - 1) / ns;
    const int n_items = lane < p.H ? ns * n_tiles : 0;
    int rank = 0;
    for (int i = 0; i < p.H; ++i) {
      const int other = __shfl_sync(0xffffffffu, per, i);
      rank += (other > per || (other == per && i < lane)) ? 1 : 0;
    }
    int start = 0;
    for (int i = 0; i < p.H; ++i) {
      const int r_i = __shfl_sync(0xffffffffu, rank, i), n_i = __shfl_sync(0xffffffffu, n_items, i);
      if (r_i < rank) start += n_i;
    }
    const int lin = static_cast<int>(blockIdx.x);  // (one-dimensional grid of nsm + H * n_tiles CTAs: the
                                                   // balance rule never makes more parts than that)
    const unsigned hit = __ballot_sync(0xffffffffu, lane < p.H && lin >= start && lin < start + n_items);
    if (hit == 0u) return;  // beyond the last real work item
    h = __ffs(hit) - 1;
    const int local = lin - __shfl_sync(0xffffffffu, start, h);
    part = local / n_tiles;
    tile = local % n_tiles;
  }
  const int row0 = tile * kTileM;
  const int g = p.group_tokens > 0 ? row0 / p.group_tokens : 0;
  const int32_t* sel = p.sel_idx + (static_cast<size_t>(h) * p.n_groups + g) * p.kcap;
  int cnt = p.do_sparse ? p.sel_cnt[static_cast<size_t>(h) * p.n_groups + g] : 0;
  cnt = max(0, min(cnt, min(p.kcap, p.n_blocks)));  // never more blocks than the history holds
  // A long list is split over the CTAs (tile, head, 0 .. nsplit - 1): each takes a run of whole
  // two-page steps; CTAs beyond nsplit leave before they set anything up.
  int nsplit = 1;
  if (SPLIT && p.max_splits > 1) {
    const int steps_total = (cnt + 1) / 2;
    nsplit = parts_of(steps_total, balance);
    const int steps_per = (steps_total + nsplit - 1) / nsplit;
    if (part >= nsplit) return;
    if (nsplit > 1) {
      const int b_lo = 2 * part * steps_per;
      const int b_hi = min(cnt, 2 * (part + 1) * steps_per);
      sel += b_lo;
      cnt = b_hi - b_lo;
    }
  }
  const int slot = (tile * p.H + h) * p.max_splits + part;  // this CTA's partial-result slot
  // steps of the compressed segment (LINF), then of the selected pages
  const int lf_pages = LINF ? p.lf_pages : 0;
  const int nA = (lf_pages + 1) / 2;
  const int nsteps = nA + (cnt + 1) / 2;
  // pages of step j (1 or 2) and whether it belongs to the compressed segment
  auto in_a = [&](int j) -> bool { return LINF && j < nA; };
  auto pages_of = [&](int j) -> int { return in_a(j) ? min(2, lf_pages - 2 * j) : min(2, cnt - 2 * (j - nA)); };

  if (SPLIT) setup();
  const uint32_t tmem = bars->tmem_base;

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

  if (warp < 4) {
    // Register budget: the CTA is allocated 168 x 384 registers.  The 128 threads here give back
    // 168 - 56 each (14336), exactly what the 256 softmax threads take to reach 224 (kSoftmaxRegs);
    // a split that asks for more than is given back would block at setmaxnreg.inc for ever.
    static_assert(128 * (168 - 56) >= 256 * (kSoftmaxRegs - 168), "setmaxnreg.inc would never be satisfied");
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
#pragma unroll 1
    for (int attempt = 0; attempt < 2; ++attempt) {
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
        auto page_row = [&](int idx) -> int32_t {
          int blk = sel[idx];
          if (blk < 0 || blk >= p.n_blocks) {  // never follow a bad index into the pool
            atomicCAS(p.status, 0, kDevBounds);
            blk = 0;
          }
          return (p.page_table[blk] * p.H + h) * kBlock;
        };
        auto load_kv = [&](int j, bool is_k) -> bool {
          const int s = j % kStages;
          const uint32_t ph = (j / kStages) & 1;
          const int npg = pages_of(j);
          const bool seg_a = in_a(j);
          uint64_t* full = is_k ? &bars->k_full[s] : &bars->v_full[s];
          uint64_t* empty = is_k ? &bars->k_empty[s] : &bars->v_empty[s];
          uint8_t* dst = smem + (is_k ? L::kK : L::kV) + s * L::kTile;
          const void* tm = seg_a ? (is_k ? static_cast<const void*>(&tm_kc) : static_cast<const void*>(&tm_vc))
                                 : (is_k ? static_cast<const void*>(&tm_k) : static_cast<const void*>(&tm_v));
          int32_t y[2] = {0, 0};
          for (int pg = 0; pg < npg; ++pg)
            y[pg] = seg_a ? (p.lf_table[2 * j + pg] * p.H + h) * kBlock : page_row(2 * (j - nA) + pg);
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
        for (int j = 0; j < min(NSB, nsteps) && ok; ++j) ok = load_kv(j, true);
#pragma unroll 1
        for (int j = 0; j < nsteps && ok; ++j) {
          ok = load_kv(j, false);
          if (ok && j + NSB < nsteps) ok = load_kv(j + NSB, true);
        }
        if (ok && p.do_linear && !LINF) {
          // hi and lo halves of the D x D state ride the V ring as two more "steps"
          for (int hl = 0; hl < 2 && ok; ++hl) {
            const int j = nsteps + hl;
            const int s = j % kStages;
            const uint32_t ph = (j / kStages) & 1;
            ok = wait_bar(&bars->v_empty[s], ph ^ 1, bars, p.status);
            if (!ok) break;
            const int rbase = ((h * 2 + p.state_slot) * 2 + hl) * D;
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
    } else if (warp == 2 && attempt == 0) {
      // ================================================================= L2 look-ahead
      // The tiles of a (head, group) walk through the same list at about the same time.  Each of
      // them asks a slice of the list (entries tile-in-group, + tiles-per-group, ...) into L2 when
      // it starts, so that between them the whole list is on its way long before the rings reach it.
      if (!SPLIT && p.k_pool != nullptr && elect_one_sync()) {  // (split tiles: measured slower with it)
        const int n_tiles = p.n_tiles;
        const int tpg = p.group_tokens > 0 ? max(1, p.group_tokens / kTileM) : n_tiles;  // tiles per group
        for (int e = kStages * 2 + tile % tpg; e < cnt; e += tpg) {
          const int blk = sel[e];
          if (blk < 0 || blk >= p.n_blocks) continue;
          const size_t off = (static_cast<size_t>(p.page_table[blk]) * p.H + h) * (kBlock * D * 2);
          bulk_prefetch_l2(p.k_pool + off, kBlock * D * 2);
          bulk_prefetch_l2(p.v_pool + off, kBlock * D * 2);
        }
      }
    } else if (warp == 1) {
      // ================================================================= MMA issuer
      if (elect_one_sync()) {
        constexpr uint32_t kHiSw = desc_hi_sw128(1024);
        const uint32_t q_lo = desc_lo_sw128(smem_u32(smem + L::kQ), 16);
        bool ok = wait_bar(&bars->q_full, 0, bars, p.status);
        tc_fence_after();
        auto issue_qk = [&](int j) -> bool {
          const int s = j % kStages;
          if (!wait_bar(&bars->k_full[s], (j / kStages) & 1, bars, p.status)) return false;
          tc_fence_after();
          const uint32_t k_lo = desc_lo_sw128(smem_u32(smem + L::kK + s * L::kTile), 16);
          const uint32_t d_tmem = tmem + kColSb + 128 * (j % NSB);
          if (pages_of(j) >= 2) {
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
          tc_commit(&bars->s_full[j % NSB]);
          return true;
        };
        for (int j = 0; j < min(NSB, nsteps) && ok; ++j) ok = issue_qk(j);
#pragma unroll 1
        for (int j = 0; j < nsteps && ok; ++j) {
          const int s = j % kStages;
          const int b = j % NSB;
          ok = wait_bar(&bars->p_full[b], (j / NSB) & 1, bars, p.status);
          if (!ok) break;
          ok = wait_bar(&bars->v_full[s], (j / kStages) & 1, bars, p.status);
          if (!ok) break;
          tc_fence_after();
          constexpr uint32_t idesc = idesc_bf16_f32(128, D, 0, 1);
          const uint32_t v_lo = desc_lo_sw128(smem_u32(smem + L::kV + s * L::kTile), L::kHalf);
          const uint32_t o_acc = tmem + (in_a(j) ? kColLn : kColO);  // each segment has its accumulator
          const uint32_t p_op = tmem + kColSb + 128 * b;
          const uint32_t acc0 = (j > 0 && !(LINF && j == nA)) ? 1u : 0u;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            tc_mma_ts_lo(o_acc, p_op + kk * 8, v_lo + kk * 128, kHiSw, idesc, kk > 0 ? 1u : acc0);
          if (pages_of(j) >= 2) {
#pragma unroll
            for (int kk = 4; kk < 8; ++kk)
              tc_mma_ts_lo(o_acc, p_op + kk * 8, v_lo + kk * 128, kHiSw, idesc, 1u);
          }
          tc_commit(&bars->v_empty[s]);
          tc_commit(&bars->pv_done);
          // the scores of step j+3 overwrite the P just consumed: issued after the P V above,
          // the tensor pipe runs them in order
          if (j + NSB < nsteps) ok = issue_qk(j + NSB);
        }
        if (ok) tc_commit(&bars->o_done);
        if (ok && p.do_linear && !LINF) {
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
              tc_mma_ts_lo(tmem + kColLn, tmem + kColPhi + kk * 8, b_lo + kk * 128, kHiSw, idesc,
                           (hl > 0 || kk > 0) ? 1u : 0u);
            tc_commit(&bars->v_empty[s]);
          }
          if (ok) tc_commit(&bars->lin_done);
        }
      }
    }
      if (!end_of_attempt()) break;
      safe = true;
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
#pragma unroll 1
    for (int attempt = 0; attempt < 2; ++attempt) {
      // ================================================================= softmax groups + epilogue
      const int grp = (warp - 4) >> 2;  // group g takes the steps j = g (mod 2)
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
      float l_a = 0.f;    // LINF: row sum of the compressed segment (l then counts the selected pages)
      bool in_b = false;  // LINF: this thread has entered the second segment
      const int64_t lf_tokens = static_cast<int64_t>(lf_pages) * kBlock;
      bool ok = true;
      const int first = safe ? (grp == 0 ? 0 : nsteps) : grp;
      const int stride = safe ? 1 : kGroups;

      // ---- linear branch operands, prepared before the loop
      constexpr int HC = D / 2;
      const bool epi = grp < 2;
      const int cbase = (grp & 1) * HC;
      float den_part = 0.f, den_part2 = 0.f;
      uint32_t fr[HC / 2];
      if (ok && p.do_linear && epi && !LINF) {
        // phi(q) of this thread's row for its half of the dims (bf16 A operand of the linear
        // MMA) and the partial denominator phi(q) . z -- computed up front, while the first scores are on their way,
        // and kept in registers until the epilogue
        ok = __all_sync(0xffffffffu, wait_bar(&bars->q_full, 0, bars, p.status));
        const uint8_t* qrow = smem + L::kQ + r * 128;
        const float exp_part = p.relu ? 0.f : 1.f;  // relu drops the exponential part of the map
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
            const uint32_t pk = pack_bf16(phi_q(__uint_as_float(qw[i] << 16), exp_part), phi_q(__uint_as_float(qw[i] & 0xffff0000u), exp_part));
            fr[c16 * 4 + i] = pk;
            // the denominator uses the rounded values the MMA will see
            den_part = fmaf(__uint_as_float(pk << 16), z[2 * i], den_part);
            den_part2 = fmaf(__uint_as_float(pk & 0xffff0000u), z[2 * i + 1], den_part2);
          }
        }
        den_part += den_part2;
      }

      // block ids of the next step are fetched one step ahead, off the critical path
      // (compressed segment: its pages in order; selected pages: the list)
      auto blocks_of = [&](int j, int& b0, int& b1) {
        if (in_a(j)) {
          b0 = 2 * j;
          b1 = 2 * j + 1;
        } else {
          const int e = 2 * (j - nA);
          b0 = sel[e];
          b1 = (e + 1 < cnt) ? sel[e + 1] : 0;
        }
      };
      int nb0 = 0, nb1 = 0;
      if (first < nsteps) blocks_of(first, nb0, nb1);
#pragma unroll 1
      for (int j = first; j < nsteps; j += stride) {
        int blk0 = nb0, blk1 = nb1;
        if (j + stride < nsteps) blocks_of(j + stride, nb0, nb1);
        // segment of this step: the compressed rows are all visible and have their own reference
        const bool seg_a = in_a(j);
        if (LINF && !seg_a && !in_b) {
          in_b = true;
          l_a = l;
          l = 0.f;
          m_used = -INFINITY;
        }
        const int jj = j - (seg_a ? 0 : nA);      // step inside its segment
        const int seg = (LINF && !seg_a) ? 1 : 0;  // which reference array / barrier
        const bool seg_first = jj == 0;
        const int seg_blocks = seg_a ? lf_pages : p.n_blocks;
        const int64_t seg_vis = seg_a ? lf_tokens : vis_end;
        const int64_t seg_tile_vis = seg_a ? lf_tokens : tile_vis_end;
        const uint32_t o_seg = seg_a ? tmem + lane_off + kColLn : o_tmem;
        const int b = j % NSB;
        const uint32_t s_tmem = tmem + lane_off + kColSb + 128 * b;
        ok = __all_sync(0xffffffffu, wait_bar(&bars->s_full[b], (j / NSB) & 1, bars, p.status));
        if (!ok) break;
        tc_fence_after();
        uint32_t cbuf[2][32];  // two 32-column chunks of the score row in flight
        // the first chunk is requested at once: its latency runs under the bookkeeping below
        // (the steps that look for the row maximum first issue their own loads)
        const bool early_ld = !(safe || seg_first);
        if (early_ld) tmem_ld32(s_tmem, cbuf[0]);
        const int npg = pages_of(j);
        const int n = npg * kBlock;
        if (blk0 < 0 || blk0 >= seg_blocks) blk0 = 0;
        if (blk1 < 0 || blk1 >= seg_blocks) blk1 = 0;
        const int64_t last_blk = blk0 > blk1 ? blk0 : blk1;
        const bool need_mask = (n != 128) || (last_blk * kBlock + kBlock > seg_tile_vis);
        // visible keys per page: columns [0, lim) of the page's 64
        int lim0 = kBlock, lim1 = kBlock;
        if (need_mask) {
          lim0 = static_cast<int>(max64(0, min64(kBlock, seg_vis - static_cast<int64_t>(blk0) * kBlock)));
          lim1 = npg > 1 ? static_cast<int>(max64(0, min64(kBlock, seg_vis - static_cast<int64_t>(blk1) * kBlock))) : 0;
        }
        const int nchunks = n / 32;
        if (safe || seg_first) {
          // the reference needs the row maximum first: a pass over the score row in chunks
          float mxa = -INFINITY, mxb = -INFINITY;
          // (the fixed reference of the fast pass only has to be near the row maximum: an unmasked
          // first step takes it from its first 32 columns)
          const int nmax = (safe || need_mask) ? nchunks : 1;
          tmem_ld32(s_tmem, cbuf[0]);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            if (c < nmax) {
              tc_wait_ld();
              if (c + 1 < nmax) tmem_ld32(s_tmem + 32 * (c + 1), cbuf[(c + 1) & 1]);
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
            bars->mref[seg][r] = t_ref;
            mbar_arrive(&bars->mref_ready[seg]);
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
              // (at the first step of the second segment nothing is rescaled: factor is 1)
              ok = __all_sync(0xffffffffu, wait_bar(&bars->pv_done, (j - 1) & 1, bars, p.status));
              if (!ok) break;
              tc_fence_after();
              if (__any_sync(0xffffffffu, factor != 1.f)) {
#pragma unroll 1
                for (int c0 = 0; c0 < D; c0 += 32) {
                  uint32_t o[32];
                  tmem_ld32(o_seg + c0, o);
                  tc_wait_ld();
#pragma unroll
                  for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
                  tmem_st32(o_seg + c0, o);
                }
                tc_wait_st();
              }
            }
            t_ref = (m_used == -INFINITY) ? 0.f : m_used * sl2;
          }
        } else if (jj < kGroups) {
          // first step of the other group in this segment (fast pass): take the reference the
          // segment's first step fixed
          ok = __all_sync(0xffffffffu, wait_bar(&bars->mref_ready[seg], 0, bars, p.status));
          if (!ok) break;
          t_ref = bars->mref[seg][r];
        }
        // exponentials in four chunks of 32 columns: the load of the next chunk and the store of
        // the previous P chunk run under the arithmetic of the current one
        const float nt = -t_ref;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};  // independent partial row sums
        if (!early_ld) tmem_ld32(s_tmem, cbuf[0]);
        if (nchunks == 4 && !need_mask) {
          // full, unmasked step (the usual case): ONE software pipeline over the 128 columns --
          // scale-and-shift of column i, exponential of column i - LAG, row sum and bf16 pack of
          // column i - 2 LAG -- that does not drain at the chunk boundaries; the TMEM load of the next
          // chunk is issued when the pipeline enters a chunk, the P store when it leaves one
          constexpr int LAG = kExpLag;
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
            // software pipeline over the chunk's 32 columns: scale-and-shift of column i, the
            // exponential of column i - LAG and the row sum / bf16 pack of column i - LAG - LAG2 are
            // issued next to each other, so that the FMA-pipe work fills the issue slots between
            // two exponentials (the SFU takes one warp instruction per 8 cycles)
            float y[32];
            uint32_t pk[16];
            constexpr int LAG = kExpLag;
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
            tmem_st16(s_tmem + 16 * c, pk);
          }
        }
        {
          const float lstep = (acc[0] + acc[1]) + (acc[2] + acc[3]);
          l += lstep;
          // a weight far above the fixed reference: finite here, but the tile is redone safely
          if (!safe && !(lstep <= kRedoSum)) bars->redo = 1;
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(&bars->p_full[b]);
      }

      // ---------------------------------------------------------------- epilogue
      // (this group's columns of the output row: group 0 -> [0, D/2), group 1 -> [D/2, D))
      if (ok && nsteps > 0) {
        ok = __all_sync(0xffffffffu, wait_bar(&bars->o_done, 0, bars, p.status));
        tc_fence_after();
      }
      if (LINF && !in_b) {  // a thread that saw no step of the second segment
        l_a = l;
        l = 0.f;
      }
      if (ok && p.do_linear && epi && !LINF) {
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
      stats[(grp * 128 + r) * 4 + 0] = l;
      stats[(grp * 128 + r) * 4 + 1] = LINF ? l_a : den_part;  // LINF: the denominator is the compressed segment's row sum
      named_bar_sync(1, 128 * kGroups);
      float lsum = 0.f, den = 0.f;
#pragma unroll
      for (int gg = 0; gg < kGroups; ++gg) {
        lsum += stats[(gg * 128 + r) * 4 + 0];
        den += stats[(gg * 128 + r) * 4 + 1];
      }
      float inv_l = (nsteps > nA && lsum > 0.f) ? 1.f / lsum : 0.f;
      const bool has_o = nsteps > nA;                       // the selected pages wrote an accumulator
      const bool has_lin = LINF ? nA > 0 : p.do_linear != 0;  // the linear branch wrote one
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
      if (ok && p.do_linear && epi && !LINF) {
        ok = __all_sync(0xffffffffu, wait_bar(&bars->lin_done, 0, bars, p.status));
        tc_fence_after();
      }
      // The output tile is staged in the Q tile's shared memory.  A tile with no step and no linear
      // branch has not looked at Q at all: its TMA load may still be in flight and must land first.
      if (ok && epi && nsteps == 0 && (!p.do_linear || LINF))
        ok = __all_sync(0xffffffffu, wait_bar(&bars->q_full, 0, bars, p.status));
      if (ok && epi && do_output) {  // warp-uniform: the TMEM loads below are warp-collective
        const bool wr = row < p.n_q;  // rows past the end of the chunk compute but never store
        float lin_den = den;
        const float* lnum = nullptr;
        if (wr && p.do_linear && p.lin_num != nullptr) {
          lnum = p.lin_num + (static_cast<size_t>(row) * p.H + h) * D;
          lin_den += p.lin_den[static_cast<size_t>(row) * p.H + h];
        }
        // (relu: a row may have no weight at all, hence 1e-6 in its denominator; 0 / 1e-6 = 0)
        const float den_eps = lin_den + ((!LINF && p.relu) ? 1e-6f : 0.f);
        const float inv_den = (p.do_linear && den_eps > 0.f) ? 1.f / den_eps : 0.f;
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
          // no gates, no causal partials, no external linear output, no merge: 32 columns per trip
          const float il = has_o ? inv_l : 0.f, id = has_lin ? inv_den : 0.f;
#pragma unroll 1
          for (int c0 = cbase; c0 < cbase + HC; c0 += 32) {
            uint32_t oa[32], ln[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) oa[i] = ln[i] = 0u;
            if (has_o) tmem_ld32(o_tmem + c0, oa);
            if (has_lin) tmem_ld32(tmem + lane_off + kColLn + c0, ln);
            tc_wait_ld();
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 32; i += 2)
              pk[i >> 1] = pack_bf16(fmaf(__uint_as_float(oa[i]), il, __uint_as_float(ln[i]) * id),
                                     fmaf(__uint_as_float(oa[i + 1]), il, __uint_as_float(ln[i + 1]) * id));
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              const int cc = (c0 >> 3) + q4;  // 16-byte chunk of the row
              *reinterpret_cast<uint4*>(smem + L::kQ + (cc >> 3) * L::kHalf + r * 128 + (((cc & 7) ^ (r & 7)) << 4)) =
                  make_uint4(pk[4 * q4], pk[4 * q4 + 1], pk[4 * q4 + 2], pk[4 * q4 + 3]);
            }
          }
        }
        // rolled on purpose: 16 columns per trip keeps this once-per-tile code small
#pragma unroll 1
        for (int c0 = cbase; c0 < (plain ? cbase : cbase + HC); c0 += 16) {
          uint32_t oa[16], ln[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) oa[i] = ln[i] = 0u;
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
          if (has_lin) tmem_ld16(tmem + lane_off + kColLn + c0, ln);
          tc_wait_ld();
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
              const float olin = has_lin ? (__uint_as_float(ln[i + e]) + ladd[i + e]) * inv_den
                                             : ladd[i + e];  // 0 unless an external linear output is given
              res[e] = fmaf(wl[i + e], olin, ws[i + e] * osp);
            }
            packed[i >> 1] = pack_bf16(res[0], res[1]);
          }
          }
          // stage the row into the Q tile's shared memory (dead by now; each thread touches only
          // its own row) in the 128-byte-swizzled layout the output tensor map expects
          {
            const int cc = c0 >> 3;  // 16-byte chunk of the row
            uint8_t* srow = smem + L::kQ + (cc >> 3) * L::kHalf + r * 128;
            *reinterpret_cast<uint4*>(srow + (((cc & 7) ^ (r & 7)) << 4)) =
                make_uint4(packed[0], packed[1], packed[2], packed[3]);
            *reinterpret_cast<uint4*>(srow + ((((cc + 1) & 7) ^ (r & 7)) << 4)) =
                make_uint4(packed[4], packed[5], packed[6], packed[7]);
          }
        }
      }
      // both epilogue groups have staged their columns: one elected thread stores the tile
      // (rows past the end of the chunk are clipped by the tensor map)
      fence_proxy_async_smem();
      named_bar_sync(2, 128 * kGroups);
      if (ok && do_output && warp == 4) {
        if (elect_one_sync()) {
          for (int dh = 0; dh < DH; ++dh) tma_store_3d(&tm_out, smem + L::kQ + dh * L::kHalf, dh * 64, h, row0);
          tma_store_commit();
          tma_store_wait_read();  // the tile must stay in shared memory until it has been read
        }
      }
      if (!end_of_attempt()) break;
      safe = true;
    }
  }

  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}


cudaError_t forward_init() {
  cudaError_t e = cudaFuncSetAttribute(hsa_forward_kernel<128, false, false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<128>::kTotal);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(hsa_forward_kernel<128, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Smem<128>::kTotal);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(hsa_forward_kernel<128, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Smem<128>::kTotal);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(hsa_forward_kernel<64, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Smem<64>::kTotal);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(hsa_forward_kernel<64, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Smem<64>::kTotal);
  return e;
}

cudaError_t launch_forward(const FwdParams& p_in, int D, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                           const CUtensorMap& tm_v, const CUtensorMap& tm_state, const CUtensorMap& tm_out,
                           cudaStream_t st, const CUtensorMap* tm_kc, const CUtensorMap* tm_vc) {
  const int n_tiles = (p_in.n_q + kTileM - 1) / kTileM;
  FwdParams p = p_in;
  p.n_tiles = n_tiles;
  const bool split = p.max_splits > 1;
  const bool linf = p.lf_table != nullptr;
  if (linf && (split || D != 128 || !tm_kc || !tm_vc)) return cudaErrorInvalidValue;
  // One list per head and few heads: the split kernel ranks the heads itself and walks a
  // one-dimensional grid longest lists first; its balance rule makes at most nsm + H * n_tiles parts.
  p.remap = split && p.n_groups == 1 && p.H <= 32;
  dim3 grid(n_tiles, p.H, split ? p.max_splits : 1);
  if (p.remap) grid = dim3(p.nsm + p.H * n_tiles);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = D == 128 ? Smem<128>::kTotal : Smem<64>::kTotal;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // (kernels without the compressed segment never look at the last two maps)
  const CUtensorMap& kc = linf ? *tm_kc : tm_k;
  const CUtensorMap& vc = linf ? *tm_vc : tm_v;
  if (D == 128) {
    if (linf) return cudaLaunchKernelEx(&cfg, hsa_forward_kernel<128, false, true>, tm_q, tm_k, tm_v, tm_state, tm_out, kc, vc, p);
    if (split) return cudaLaunchKernelEx(&cfg, hsa_forward_kernel<128, true, false>, tm_q, tm_k, tm_v, tm_state, tm_out, kc, vc, p);
    return cudaLaunchKernelEx(&cfg, hsa_forward_kernel<128, false, false>, tm_q, tm_k, tm_v, tm_state, tm_out, kc, vc, p);
  }
  if (split) return cudaLaunchKernelEx(&cfg, hsa_forward_kernel<64, true, false>, tm_q, tm_k, tm_v, tm_state, tm_out, kc, vc, p);
  return cudaLaunchKernelEx(&cfg, hsa_forward_kernel<64, false, false>, tm_q, tm_k, tm_v, tm_state, tm_out, kc, vc, p);
}

}  // namespace hsa
