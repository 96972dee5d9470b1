// hsa_select_blocks kernels: mean query per group, pooled block scores
//   s[h,g,b] = mean_q(g) . (Ksum[h,b] / cnt_b) * scale
// and an exact per-(head, group) top-k by radix select, all on the device:
// query partial sums -> scores (many CTAs) -> top-k (one block of 256 threads per head and group).
// The stages run in one of three forms (see launch_select): a kernel for the query sums followed
// by one thread-block cluster per head, one cooperative launch with two grid barriers, or three
// launches.
#include <cuda_bf16.h>

#include <cmath>
#include <mutex>

#include "grid_sync.cuh"
#include "hsa_internal.h"

namespace hsa {

// The stages below are written for a block of 256 threads.  That block is either a whole CTA (tid =
// threadIdx.x, barrier 0) or one of several sub-blocks of a larger CTA, each with its own named
// barrier (the cluster form of the fused kernel runs three of them per CTA).
struct Blk {
  int tid;  // 0..255 inside the block
  int bar;  // named barrier of the block
};
__device__ __forceinline__ void blk_sync(const Blk& blk) {
  asm volatile("bar.sync %0, 256;" ::"r"(blk.bar) : "memory");
}

// ---------------------------------------------------------------------------------------
// Stage 1: column sums of q over one 128-token tile and one head -> qpart[tile][h][D].
// ---------------------------------------------------------------------------------------
template <int D>
__device__ __forceinline__ void qsum_item(const Blk& blk, const SelectArgs& a, int tile, int h, float (*red)[D]) {
  constexpr int CH = D / 8;
  constexpr int RP = 256 / CH;
  const int c8 = blk.tid % CH, rg = blk.tid / CH;
  const int t_hi = min(a.n_q, tile * kTileM + kTileM);
  float acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.f;
  // all of a thread's rows are requested before any is consumed (independent loads in flight)
  constexpr int NR = kTileM / RP;
  uint4 rows[NR];
#pragma unroll
  for (int i = 0; i < NR; ++i) {
    const int t = tile * kTileM + rg + i * RP;
    rows[i] = make_uint4(0, 0, 0, 0);
    if (t < t_hi)
      rows[i] = *reinterpret_cast<const uint4*>(a.q + static_cast<size_t>(t) * a.tok_stride +
                                                static_cast<size_t>(h) * a.head_stride + c8 * 8);
  }
#pragma unroll
  for (int i = 0; i < NR; ++i) {
    const __nv_bfloat162* q2 = reinterpret_cast<const __nv_bfloat162*>(&rows[i]);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(q2[e]);
      acc[2 * e] += f.x;
      acc[2 * e + 1] += f.y;
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) red[rg][c8 * 8 + i] = acc[i];
  blk_sync(blk);
  if (blk.tid < D) {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < RP; ++r) s += red[r][blk.tid];
    a.qpart[(static_cast<size_t>(tile) * a.H + h) * D + blk.tid] = s;
  }
}

template <int D>
__global__ void __launch_bounds__(256) qsum_partial_kernel(SelectArgs a) {
  __shared__ float red[256 / (D / 8)][D];
  // (no-ops unless launched with programmatic stream serialization: wait for the kernel before this
  // one, let the kernel behind this one be scheduled early -- it waits for this grid's end itself)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  qsum_item<D>(Blk{static_cast<int>(threadIdx.x), 0}, a, blockIdx.x, blockIdx.y, red);
}

__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // ascending with the float order
}

__device__ __forceinline__ int block_exclusive_scan(const Blk& blk, int v, int* warp_sums, int* total) {
  // 256 threads; returns the exclusive prefix of v over blk.tid and the block total
  const int lane = blk.tid & 31, warp = blk.tid >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  blk_sync(blk);
  if (lane == 31) warp_sums[warp] = incl;
  blk_sync(blk);
  int base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < 8; ++w) {
    const int s = warp_sums[w];
    if (w < warp) base += s;
    tot += s;
  }
  *total = tot;
  return base + incl - v;
}

// ---------------------------------------------------------------------------------------
// Candidates.  A candidate is a run of consecutive pages that is scored and selected as one:
// pages [0, p0) form "inter-chunk" candidates of `inter_pages` pages each (the last one may be
// short), pages [p0, nblk) are "intra-chunk" candidates of one page each.  The default
// (inter_pages = 1, p0 = nblk) makes every page its own candidate.
// ---------------------------------------------------------------------------------------
struct CandGeom {
  int nblk, p0;
  int ip;      // pages per inter-chunk candidate
  int ni, nc;  // inter-chunk candidates, all candidates
};
// MIXED = false is the plain case, known at compile time: one page per candidate, no intra part
template <bool MIXED>
__device__ __forceinline__ CandGeom cand_geom(const SelectArgs& a) {
  CandGeom g;
  g.nblk = static_cast<int>((a.n_tokens + kBlock - 1) / kBlock);
  if (!MIXED) {
    g.ip = 1;
    g.p0 = g.ni = g.nc = g.nblk;
    return g;
  }
  g.ip = a.inter_pages > 1 ? a.inter_pages : 1;
  g.p0 = (a.intra_first_page1 > 0 && a.intra_first_page1 <= g.nblk) ? static_cast<int>(a.intra_first_page1 - 1) : g.nblk;
  g.ni = (g.p0 + g.ip - 1) / g.ip;
  g.nc = g.ni + (g.nblk - g.p0);
  return g;
}
template <bool MIXED>
__device__ __forceinline__ int cand_first_page(const CandGeom& g, int c) {
  if (!MIXED) return c;
  return c < g.ni ? c * g.ip : g.p0 + (c - g.ni);
}
template <bool MIXED>
__device__ __forceinline__ int cand_pages(const CandGeom& g, int c) {
  if (!MIXED) return 1;
  return c < g.ni ? min(g.ip, g.p0 - c * g.ip) : 1;
}
// candidates whose first token is at or before position p_last (they form a prefix)
template <bool MIXED>
__device__ __forceinline__ int cand_visible(const CandGeom& g, int64_t p_last) {
  if (p_last < 0) return 0;
  const int pg = static_cast<int>(min64(p_last / kBlock, g.nblk));  // page that holds p_last
  if (!MIXED) return min(g.nblk, pg + 1);
  if (pg < g.p0) return min(g.ni, pg / g.ip + 1);
  return min(g.nc, g.ni + (pg - g.p0) + 1);
}

// ---------------------------------------------------------------------------------------
// Stage 2: pooled scores.  grid (ceil(nblk/32), n_groups, H); one warp per block, four blocks
// per warp.  The mean query of the group is rebuilt from the tile partials in fp64 (fixed
// order), the dot product runs in fp64 and is rounded once to the fp32 sort key.
// ---------------------------------------------------------------------------------------
constexpr int kScoreBlocksPerCta = 32;

// The key sums one item needs, per lane: candidates chunk * 32 + i * 8 + warp, dims lane * PER .. + PER - 1
// of at most two pages each.  They depend on nothing the kernel computes, so the fused kernel asks
// for those of its first item before the first grid barrier and lets their latency run under it.
template <int D, bool MIXED>
struct ScoreOperands {
  static constexpr int PER = D / 32, NB = kScoreBlocksPerCta / 8, NP = MIXED ? 2 : 1;
  float kv[NB][NP][PER];
};
template <int D, bool MIXED>
__device__ __forceinline__ void scores_load(const Blk& blk, const SelectArgs& a, int chunk, int h, ScoreOperands<D, MIXED>& op) {
  using O = ScoreOperands<D, MIXED>;
  const int lane = blk.tid & 31, warp = blk.tid >> 5;
  const CandGeom cg = cand_geom<MIXED>(a);
#pragma unroll
  for (int i = 0; i < O::NB; ++i) {
    const int c = chunk * kScoreBlocksPerCta + i * 8 + warp;
    const int fp = c < cg.nc ? cand_first_page<MIXED>(cg, c) : 0;
    const int np = c < cg.nc ? cand_pages<MIXED>(cg, c) : 0;
#pragma unroll
    for (int pg = 0; pg < O::NP; ++pg)
#pragma unroll
      for (int e = 0; e < O::PER; ++e)
        op.kv[i][pg][e] =
            pg < np ? a.ksum[(static_cast<size_t>(h) * a.max_pages + fp + pg) * D + lane * O::PER + e] : 0.f;
  }
}

// rebuild = false: qs[0, D) still holds the mean query of this (group, head) from the item before;
// loaded = true: `op` already holds this item's key sums; keys_cluster_addr != 0: where the keys go
// instead of the workspace
template <int D, bool MIXED>
__device__ __forceinline__ void scores_item(const Blk& blk, const SelectArgs& a, int chunk, int g, int h, double* qs,
                                            ScoreOperands<D, MIXED>& op, bool rebuild = true, bool loaded = false,
                                            uint32_t keys_cluster_addr = 0) {
  const int lane = blk.tid & 31, warp = blk.tid >> 5;
  const int gtok = a.group_tokens > 0 ? a.group_tokens : a.n_q;
  const int q_lo = g * gtok, q_hi = min(a.n_q, q_lo + gtok);
  if (!loaded) scores_load<D, MIXED>(blk, a, chunk, h, op);  // in flight while the mean query is rebuilt
  if (rebuild) {
    // 256 / D threads per column, each summing an interleaved subset of the tile partials with
    // up to 20 loads in flight (one round trip for a chunk of up to 40 tiles at head_dim 128); the subsets are then added in a fixed order
    constexpr int WAYS = 256 / D;
    constexpr int kInFlight = 20;
    const int col = blk.tid % D, way = blk.tid / D;
    const int tile_lo = q_lo / kTileM, tile_hi = (q_hi + kTileM - 1) / kTileM;
    double s = 0.0;
    for (int t0 = tile_lo + way; t0 < tile_hi; t0 += kInFlight * WAYS) {
      float v[kInFlight];
#pragma unroll
      for (int i = 0; i < kInFlight; ++i)
        v[i] = (t0 + i * WAYS < tile_hi) ? __ldcg(&a.qpart[(static_cast<size_t>(t0 + i * WAYS) * a.H + h) * D + col]) : 0.f;
#pragma unroll
      for (int i = 0; i < kInFlight; ++i) s += static_cast<double>(v[i]);
    }
    double* part = qs + D;  // [WAYS][D]
    part[way * D + col] = s;
    blk_sync(blk);
    if (blk.tid < D) {
      double t = 0.0;
#pragma unroll
      for (int w = 0; w < WAYS; ++w) t += part[w * D + blk.tid];
      qs[blk.tid] = t / static_cast<double>(q_hi - q_lo) * static_cast<double>(a.scale);
    }
    blk_sync(blk);  // (a mean query that was not rebuilt here is complete already: no barrier, the
                    // warps walk through their candidates independently)
  }
  constexpr int PER = D / 32;
  uint32_t* keys = a.keys + (static_cast<size_t>(h) * a.n_groups + g) * a.max_pages;
  const CandGeom cg = cand_geom<MIXED>(a);
  constexpr int NB = kScoreBlocksPerCta / 8;  // candidates per warp
  constexpr int NP = MIXED ? 2 : 1;           // pages per candidate at most
  auto& kv = op.kv;
  // this lane's part of the NB dot products (fp64), then ONE reduction for all of them: at each of
  // the first steps a lane hands half of its values to its partner and keeps the other half
  // (value i ends up in the lanes whose bits 4, 3 (NB = 4) spell i), the remaining steps add single
  // values -- NB + 2 adds and 2 NB - 2 + 3 exchanges instead of 5 adds and 5 exchanges per candidate
  static_assert(NB == 4, "the reduction below is written for four candidates per warp");
  double dot[NB];
#pragma unroll
  for (int i = 0; i < NB; ++i) {
    dot[i] = 0.0;
#pragma unroll
    for (int e = 0; e < PER; ++e)
      dot[i] += qs[lane * PER + e] * (static_cast<double>(kv[i][0][e]) + (MIXED ? static_cast<double>(kv[i][NP - 1][e]) : 0.0));
  }
  {
    // step 1 (partner lane ^ 16): lanes with bit 4 clear keep candidates 0, 1 and give 2, 3
    const bool up = (lane & 16) != 0;
    const double g0 = up ? dot[0] : dot[2], g1 = up ? dot[1] : dot[3];
    const double k0 = up ? dot[2] : dot[0], k1 = up ? dot[3] : dot[1];
    dot[0] = k0 + __shfl_xor_sync(0xffffffffu, g0, 16);
    dot[1] = k1 + __shfl_xor_sync(0xffffffffu, g1, 16);
    // step 2 (partner lane ^ 8): lanes with bit 3 clear keep the first of their two
    const bool up2 = (lane & 8) != 0;
    const double g = up2 ? dot[0] : dot[1], k = up2 ? dot[1] : dot[0];
    dot[0] = k + __shfl_xor_sync(0xffffffffu, g, 8);
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) dot[0] += __shfl_xor_sync(0xffffffffu, dot[0], o);
  }
  // lanes 0, 8, 16, 24 now hold the sums of candidates 0, 1, 2, 3 (lane bits 4, 3 = candidate: bit 4
  // chose between {0, 1} and {2, 3}, bit 3 inside the pair)
  if ((lane & 7) == 0) {
    const int i = ((lane >> 4) & 1) * 2 + ((lane >> 3) & 1);
    const int c = chunk * kScoreBlocksPerCta + i * 8 + warp;
    if (c < cg.nc) {
      const int64_t t0 = static_cast<int64_t>(cand_first_page<MIXED>(cg, c)) * kBlock;
      const int64_t cnt = min64(static_cast<int64_t>(cand_pages<MIXED>(cg, c)) * kBlock, a.n_tokens - t0);
      // a full block's mean is an exact scaling; only a partly filled block needs the division
      const double mean = cnt == kBlock ? dot[0] * (1.0 / kBlock) : dot[0] / static_cast<double>(cnt);
      uint32_t key = order_key(static_cast<float>(mean));
      if (MIXED && a.kv_pages != nullptr && c < cg.ni) {
        // every page of the candidate must lie in a retrieved KV page; key 0 marks "no candidate"
        const int pf = cand_first_page<MIXED>(cg, c), pl = pf + cand_pages<MIXED>(cg, c) - 1;
        bool in_f = false, in_l = false;
        for (int j = 0; j < a.n_kv_pages; ++j) {
          const int kp = a.kv_pages[j];
          in_f |= (pf / a.kv_page_blocks == kp);
          in_l |= (pl / a.kv_page_blocks == kp);
        }
        if (!(in_f && in_l)) key = 0u;
      }
      // cluster form: straight into the key array of the CTA that extracts the list (a
      // shared::cluster address), else into the workspace
      if (keys_cluster_addr)
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(keys_cluster_addr + 4u * static_cast<uint32_t>(c)), "r"(key) : "memory");
      else
        keys[c] = key;
    }
  }
}


// Many query groups (per-query-tile selection): the scores of one head are a small matrix product
//   scores[g][c] = sum_e qbar[g][e] * ksum[c][e]
// and plain fp64 arithmetic is a slow pipe on this GPU, so it runs on the fp64 tensor-core path
// (mma.sync m8n8k4).  One item is a chunk of 32 candidates of one head for ALL groups, so that the
// key sums are read once: warp w owns candidates 8 (w & 3) .. + 7 (their key sums sit in registers as
// the B fragments of all k-steps) and rows 8 (w >> 2) .. + 7 of each batch of 16 groups, whose mean
// queries are rebuilt in shared memory (qs: 16 rows of D + 4 doubles; the pad keeps the fragment
// loads at the two wavefronts a 256-byte access needs anyway).
constexpr int kGroupBatch = 16;

__device__ __forceinline__ void dmma_m8n8k4(double& d0, double& d1, double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(d0), "+d"(d1)
               : "d"(a), "d"(b));
}

template <int D, bool MIXED>
__device__ __forceinline__ void scores_item_groups(const Blk& blk, const SelectArgs& a, int chunk, int h, double* qs) {
  constexpr int GB = kGroupBatch, PITCH = D + 4, KS = D / 4;
  const int lane = blk.tid & 31, warp = blk.tid >> 5;
  const int gtok = a.group_tokens;  // > 0 here, a multiple of the tile height
  const CandGeom cg = cand_geom<MIXED>(a);
  const int c0 = chunk * kScoreBlocksPerCta + 8 * (warp & 3);  // this warp's eight candidates
  // B fragments: element (k = lane % 4, n = lane / 4) of every k-step = key sum of candidate
  // c0 + lane / 4 at dims 4 kk + lane % 4 (a coarse candidate's two pages are added here)
  float kb[KS];
  {
    const int c = c0 + (lane >> 2);
    const int fp = c < cg.nc ? cand_first_page<MIXED>(cg, c) : 0;
    const int np = c < cg.nc ? cand_pages<MIXED>(cg, c) : 0;
    const float* k0 = a.ksum + (static_cast<size_t>(h) * a.max_pages + fp) * D + (lane & 3);
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
      float v = np > 0 ? k0[4 * kk] : 0.f;
      if (MIXED && np > 1) v += k0[D + 4 * kk];
      kb[kk] = v;
    }
  }
  // the two candidates of this lane's accumulator columns: token counts and mask
  double inv_cnt[2];
  bool masked[2];
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int c = c0 + 2 * (lane & 3) + t;
    const int fp = c < cg.nc ? cand_first_page<MIXED>(cg, c) : 0;
    const int np = c < cg.nc ? cand_pages<MIXED>(cg, c) : 0;
    // (fp64 division is a long instruction sequence on a slow pipe: a full page's count is a power
    // of two, only a partly filled candidate needs the division)
    const int64_t cnt = max64(1, min64(static_cast<int64_t>(np) * kBlock, a.n_tokens - static_cast<int64_t>(fp) * kBlock));
    inv_cnt[t] = cnt == kBlock ? 1.0 / kBlock : 1.0 / static_cast<double>(cnt);
    masked[t] = false;
    if (MIXED && a.kv_pages != nullptr && c < cg.ni) {
      const int pl = fp + np - 1;
      bool in_f = false, in_l = false;
      for (int k = 0; k < a.n_kv_pages; ++k) {
        const int kp = a.kv_pages[k];
        in_f |= (fp / a.kv_page_blocks == kp);
        in_l |= (pl / a.kv_page_blocks == kp);
      }
      masked[t] = !(in_f && in_l);
    }
  }
  const int tiles_per_group = gtok / kTileM;
  const double mean_scale_full = static_cast<double>(a.scale) / static_cast<double>(gtok);  // all groups but a short last one
  for (int g0 = 0; g0 < a.n_groups; g0 += GB) {
    // mean queries of groups g0 .. g0 + 15 (tile sums added in ascending tile order, fp64)
    constexpr int NV = GB * D / 256;  // values per thread
    double sum[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) sum[v] = 0.0;
    for (int tt = 0; tt < tiles_per_group; ++tt) {
      float part[NV];  // independent loads first, then the adds
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const int idx = blk.tid + 256 * v;
        const int g = g0 + idx / D, col = idx % D;
        const int t = g * tiles_per_group + tt;
        part[v] = (g < a.n_groups && t * kTileM < a.n_q) ? __ldcg(&a.qpart[(static_cast<size_t>(t) * a.H + h) * D + col]) : 0.f;
      }
#pragma unroll
      for (int v = 0; v < NV; ++v) sum[v] += static_cast<double>(part[v]);
    }
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const int idx = blk.tid + 256 * v;
      const int gi = idx / D, g = g0 + gi;
      const int q_lo = g * gtok, q_hi = min(a.n_q, q_lo + gtok);
      const double ms = (q_hi - q_lo == gtok) ? mean_scale_full : static_cast<double>(a.scale) / static_cast<double>(q_hi - q_lo);
      qs[gi * PITCH + idx % D] = g < a.n_groups ? sum[v] * ms : 0.0;
    }
    blk_sync(blk);
    const int row0 = 8 * (warp >> 2);  // this warp's eight rows of the batch
    if (g0 + row0 < a.n_groups && c0 < cg.nc) {  // warp-uniform
      // A fragment: element (m = lane / 4, k = lane % 4) of every k-step
      const double* arow = qs + (row0 + (lane >> 2)) * PITCH + (lane & 3);
      double d0 = 0.0, d1 = 0.0;
#pragma unroll
      for (int kk = 0; kk < KS; ++kk) dmma_m8n8k4(d0, d1, arow[4 * kk], static_cast<double>(kb[kk]));
      // accumulator: row lane / 4 (group), columns 2 (lane % 4) and + 1 (candidates)
      const int g = g0 + row0 + (lane >> 2);
      if (g < a.n_groups) {
        uint32_t* keys = a.keys + (static_cast<size_t>(h) * a.n_groups + g) * a.max_pages;
        const int c = c0 + 2 * (lane & 3);
        if (c < cg.nc) keys[c] = masked[0] ? 0u : order_key(static_cast<float>(d0 * inv_cnt[0]));
        if (c + 1 < cg.nc) keys[c + 1] = masked[1] ? 0u : order_key(static_cast<float>(d1 * inv_cnt[1]));
      }
    }
    blk_sync(blk);
  }
}

template <int D, bool MIXED>
__global__ void __launch_bounds__(256) block_scores_kernel(SelectArgs a) {
  __shared__ double qs[D + 256];  // mean query, then the per-way partial sums
  asm volatile("griddepcontrol.wait;" ::: "memory");  // (see qsum_partial_kernel)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  ScoreOperands<D, MIXED> op;
  scores_item<D, MIXED>(Blk{static_cast<int>(threadIdx.x), 0}, a, blockIdx.x, blockIdx.y, blockIdx.z, qs, op);
}

// ---------------------------------------------------------------------------------------
// Stage 3: one CTA per (group, head): k-th largest key by a 4-pass 8-bit radix select, then an
// index-ordered compaction.  Exact ties at the threshold go to the lower block index.
// dynamic smem: uint32 keys[ncand]
// ---------------------------------------------------------------------------------------
struct TopkShared {
  int hist[256];
  int warp_sums[8];
  uint32_t prefix;
  int krem;
  int exact;  // radix select: the bin just chosen holds exactly the keys still to take
};

// The `budget` largest keys of keys[0, n) (ties at the threshold to the lower index), emitted in
// index order as the pages of candidates c0 + i; returns the number of pages emitted (whether or
// not they fitted below kcap).  All 256 threads call it; keys live in shared memory.
template <bool MIXED>
__device__ __forceinline__ int topk_range(const Blk& blk, const uint32_t* keys, int n, int budget, const CandGeom& cg, int c0,
                                          int32_t* out, int out_pos0, int kcap, TopkShared* sh, bool masked) {
  int* hist = sh->hist;
  int* warp_sums = sh->warp_sums;
  // keys equal to 0 are masked-out candidates (no finite score maps to 0): they are never chosen
  int n_eff = n;
  if (MIXED && masked) {
    int my0 = 0, tot0 = 0;
    for (int b = blk.tid; b < n; b += 256) my0 += (keys[b] == 0u);
    block_exclusive_scan(blk, my0, warp_sums, &tot0);
    blk_sync(blk);
    n_eff = n - tot0;
  }
  if (budget < 0 || budget > n_eff) budget = n_eff;
  const bool take_all = (budget >= n_eff);
  uint32_t thr = 0;
  int need_ties = 0;
  if (!take_all && budget > 0) {
    uint32_t mask = 0, prefix = 0;
    int krem = budget;
    for (int pass = 3; pass >= 0; --pass) {
      const int shift = pass * 8;
      hist[blk.tid] = 0;
      blk_sync(blk);
      for (int b = blk.tid; b < n; b += 256) {
        const uint32_t k = keys[b];
        if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 255], 1);
      }
      blk_sync(blk);
      // thread t owns bin 255 - t: an inclusive prefix over t is the count of keys in bins >= own
      const int bin = 255 - static_cast<int>(blk.tid);
      const int mine = hist[bin];
      int tot;
      const int above = block_exclusive_scan(blk, mine, warp_sums, &tot);  // keys in strictly higher bins
      if (above < krem && above + mine >= krem) {                     // exactly one thread
        sh->prefix = prefix | (static_cast<uint32_t>(bin) << shift);
        sh->krem = krem - above;  // still to take among keys matching the longer prefix
        sh->exact = (above + mine == krem);
      }
      blk_sync(blk);
      prefix = sh->prefix;
      krem = sh->krem;
      mask |= 255u << shift;
      // every key of the chosen bin is wanted: the prefix with zero low bits is a threshold that
      // all of them reach, and krem (their number) covers the ones that equal it exactly
      if (sh->exact) break;
    }
    thr = prefix;
    need_ties = krem;
  }

  // index-ordered compaction: thread t owns the contiguous range [t*per, t*per+per)
  const int per = (n + 255) / 256;
  const int lo = min(n, static_cast<int>(blk.tid) * per), hi = min(n, lo + per);
  const bool use_mask = per <= 32;  // the thread's range fits a 32-bit mask: ONE walk over the keys
  int ties_before = 0, dummy;
  uint32_t gt = 0, eq = 0;  // candidates above the threshold / equal to it, as bits of the range
  if (use_mask) {
    for (int b = lo; b < hi; ++b) {
      const uint32_t k = keys[b];
      const uint32_t bit = 1u << (b - lo);
      if (take_all) {
        if (!(MIXED && masked) || k != 0u) gt |= bit;
      } else if (budget > 0) {
        if (k > thr)
          gt |= bit;
        else if (k == thr)
          eq |= bit;
      }
    }
    if (!take_all && budget > 0) ties_before = block_exclusive_scan(blk, __popc(eq), warp_sums, &dummy);
  } else if (!take_all && budget > 0) {
    int my_ties = 0;
    for (int b = lo; b < hi; ++b) my_ties += (keys[b] == thr);
    ties_before = block_exclusive_scan(blk, my_ties, warp_sums, &dummy);
  }
  auto chosen = [&](int b, int& t) -> bool {
    if (take_all) return !(MIXED && masked) || keys[b] != 0u;
    if (budget == 0) return false;
    const uint32_t k = keys[b];
    if (k == thr) return t++ < need_ties;
    return k > thr;
  };
  // which of this thread's candidates are chosen and how many pages they hold; after the scan: emit
  int my_pages = 0;
  uint32_t picked = 0;
  if (use_mask) {
    // ties at the threshold go to the lowest indices: this thread's ties rank ties_before, + 1, ...
    int allow = need_ties - ties_before;
    uint32_t e = eq;
    while (allow > 0 && e) {
      picked |= e & (0u - e);
      e &= e - 1;
      --allow;
    }
    picked |= gt;
    if (!MIXED) {
      my_pages = __popc(picked);
    } else {
      for (uint32_t m = picked; m; m &= m - 1) my_pages += cand_pages<MIXED>(cg, c0 + lo + __ffs(m) - 1);
    }
  } else {
    int t = ties_before;
    for (int b = lo; b < hi; ++b)
      if (chosen(b, t)) my_pages += cand_pages<MIXED>(cg, c0 + b);
  }
  int total = 0;
  int pos = out_pos0 + block_exclusive_scan(blk, my_pages, warp_sums, &total);
  auto emit = [&](int b) {
    const int fp = cand_first_page<MIXED>(cg, c0 + b);
    const int np = cand_pages<MIXED>(cg, c0 + b);
    for (int pg = 0; pg < np; ++pg, ++pos)
      if (pos < kcap) out[pos] = fp + pg;
  };
  if (use_mask) {
    while (picked) {
      const int i = __ffs(picked) - 1;
      picked &= picked - 1;
      emit(lo + i);
    }
  } else {
    int t = ties_before;
    for (int b = lo; b < hi; ++b)
      if (chosen(b, t)) emit(b);
  }
  blk_sync(blk);  // hist / warp_sums are reused by the next call
  return total;
}

// keys_in_place: `keys` already holds the head's score keys (the cluster form writes them there)
template <bool MIXED>
__device__ __forceinline__ void topk_item(const Blk& blk, const SelectArgs& a, int g, int h, uint32_t* keys, TopkShared* sh,
                                          int budget, int intra_budget, bool keys_in_place = false) {
  const CandGeom cg = cand_geom<MIXED>(a);
  const int gtok = a.group_tokens > 0 ? a.group_tokens : a.n_q;
  const int q_hi = min(a.n_q, g * gtok + gtok);
  const int64_t p_last = a.q_pos0 + q_hi - 1;
  // candidates are a prefix [0, ncand): all of them, or those that start at or before the group's
  // last query position
  const int ncand = a.causal ? cand_visible<MIXED>(cg, p_last) : cg.nc;
  const uint32_t* gkeys = a.keys + (static_cast<size_t>(h) * a.n_groups + g) * a.max_pages;
  if (!keys_in_place)
    for (int b = blk.tid; b < ncand; b += 256) keys[b] = __ldcg(&gkeys[b]);
  if (blk.tid == 0) {
    sh->prefix = 0;
    sh->krem = 0;
  }
  blk_sync(blk);
  int32_t* out = a.sel_idx + (static_cast<size_t>(h) * a.n_groups + g) * a.kcap;
  // inter-chunk candidates against the head's budget, then intra-chunk ones against theirs
  const int n_inter = min(ncand, cg.ni);
  int total = topk_range<MIXED>(blk, keys, n_inter, budget, cg, 0, out, 0, a.kcap, sh, a.kv_pages != nullptr);
  if (MIXED && ncand > n_inter)
    total += topk_range<MIXED>(blk, keys + n_inter, ncand - n_inter, intra_budget, cg, cg.ni, out, total, a.kcap, sh, false);
  if (blk.tid == 0) {
    a.sel_cnt[static_cast<size_t>(h) * a.n_groups + g] = min(total, a.kcap);
    if (total > a.kcap) atomicCAS(a.status, 0, kDevBounds);
  }
}

template <bool MIXED>
__global__ void __launch_bounds__(256) topk_kernel(SelectArgs a) {
  extern __shared__ uint32_t topk_keys[];
  __shared__ TopkShared sh;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // (see qsum_partial_kernel)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int h = blockIdx.y;
  topk_item<MIXED>(Blk{static_cast<int>(threadIdx.x), 0}, a, blockIdx.x, h, topk_keys, &sh, a.budgets[h],
                   (MIXED && a.intra_budgets) ? a.intra_budgets[h] : -1);
}

// ---------------------------------------------------------------------------------------
// The three stages in ONE cooperative launch (all CTAs co-resident): query tile sums, grid
// barrier, scores, grid barrier, top-k.  Saves two launches and their drain / ramp-up.
//
// The grid barrier (device_barrier: two words in the workspace, an arrive count and a generation)
// lives entirely on the device, so a launch captured in a CUDA graph behaves the same on every
// replay, in any order with other launches.  Its wait is bounded (wait_ns): on expiry the CTA
// records a timeout in the status word and the kernel ends with every list of the call counted
// as empty.  The host clears the two words when it reads that status (hsa_device_status).
// ---------------------------------------------------------------------------------------
template <int D, bool MIXED>
__global__ void __launch_bounds__(256, 3) select_fused_kernel(SelectArgs a) {
  extern __shared__ uint32_t fused_keys[];
  // tile-sum partials / mean query / (many groups) a batch of mean queries
  constexpr int kGroupBytes = kGroupBatch * (D + 4) * 8;
  constexpr int kScratch = kGroupBytes > 256 / (D / 8) * D * 4 ? kGroupBytes : 256 / (D / 8) * D * 4;
  __shared__ __align__(16) unsigned char scratch[kScratch];
  __shared__ TopkShared sh;
  const Blk blk{static_cast<int>(threadIdx.x), 0};
  // launched as a programmatic dependent: the kernel before this one is complete from here on
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int n_tiles = (a.n_q + kTileM - 1) / kTileM;
  const int n_chunks = (cand_geom<MIXED>(a).nc + kScoreBlocksPerCta - 1) / kScoreBlocksPerCta;
  // a barrier that ran out: no list of this call can be trusted, every one is counted as empty
  auto give_up = [&]() {
    for (int it = blockIdx.x; it < a.n_groups * a.H; it += gridDim.x)
      if (threadIdx.x == 0) a.sel_cnt[it] = 0;  // it = h * n_groups + g
  };
  // one selection per head: a CTA takes a run of consecutive (head, chunk) score items; the key sums
  // of the first one are requested now, ahead of the query sums and the first barrier
  const int n_items = n_chunks * a.H;
  const int per = (n_items + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
  const int it0 = static_cast<int>(blockIdx.x) * per, it1 = min(n_items, it0 + per);
  ScoreOperands<D, MIXED> op;
  const bool ahead = a.n_groups == 1 && it0 < it1;
  if (ahead) scores_load<D, MIXED>(blk, a, it0 % n_chunks, it0 / n_chunks, op);
  for (int it = blockIdx.x; it < n_tiles * a.H; it += gridDim.x) {
    qsum_item<D>(blk, a, it % n_tiles, it / n_tiles, reinterpret_cast<float(*)[D]>(scratch));
    __syncthreads();
  }
  if (!device_barrier(a.barrier, gridDim.x, a.status, a.wait_ns)) {
    give_up();
    return;
  }
  if (a.n_groups > 1) {
    for (int it = blockIdx.x; it < n_chunks * a.H; it += gridDim.x)
      scores_item_groups<D, MIXED>(blk, a, it % n_chunks, it / n_chunks, reinterpret_cast<double*>(scratch));
  } else {
    // the mean query of a head is rebuilt from the tile partials only when the run enters the head
    int h_cur = -1;
    for (int it = it0; it < it1; ++it) {
      const int h = it / n_chunks;
      scores_item<D, MIXED>(blk, a, it % n_chunks, 0, h, reinterpret_cast<double*>(scratch), op, h != h_cur, it == it0);
      h_cur = h;
      __syncthreads();
    }
  }
  if (!device_barrier(a.barrier, gridDim.x, a.status, a.wait_ns)) {
    give_up();
    return;
  }
  // Only a few CTAs have a list to extract; the others leave now.  The kernel behind this one
  // (launched as a programmatic dependent, it waits for this grid's end before it reads a list)
  // may take their places and do its set-up meanwhile.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  for (int it = blockIdx.x; it < a.n_groups * a.H; it += gridDim.x) {
    const int h = it / a.n_groups;
    topk_item<MIXED>(blk, a, it % a.n_groups, h, fused_keys, &sh, a.budgets[h], (MIXED && a.intra_budgets) ? a.intra_budgets[h] : -1);
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------------------
// The score and list stages with the CTAs of a head forming a thread-block cluster: everything a
// head's lists need -- its scores -- is produced inside its cluster, so the synchronisation point
// between the two stages is a hardware cluster barrier (release / acquire at cluster scope) instead
// of a grid-wide barrier in global memory, and the launch needs no co-residency of the whole grid.
// The query tile sums come from qsum_partial_kernel, launched in front of this kernel (they read the
// whole chunk and want every SM; this kernel waits for them as a programmatic dependent).
// grid = H clusters of CS CTAs; a CTA holds kSubBlocks blocks of 256 threads, each of which takes
// work items of its own (slot = cluster rank * kSubBlocks + sub-block).
// ---------------------------------------------------------------------------------------
constexpr int kSubBlocks = 3;

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int D>
struct ClusterSmem {
  static constexpr int kScratch = (D + 256) * 8;  // per sub-block; together: mean query [D] + partial sums [768 / D][D], fp64
  static constexpr int kFixed = (kSubBlocks * kScratch + static_cast<int>(sizeof(TopkShared)) + 15) / 16 * 16;
};

template <int D, bool MIXED>
__global__ void __launch_bounds__(256 * kSubBlocks, 1) select_cluster_kernel(SelectArgs a, int cluster_ctas) {
  // dynamic shared memory: per sub-block scratch (mean query and its partial sums) | top-k
  // bookkeeping | the head's keys
  extern __shared__ __align__(16) unsigned char cl_smem[];
  constexpr int kScratch = ClusterSmem<D>::kScratch;
  const int sub = static_cast<int>(threadIdx.x) / 256;
  const Blk blk{static_cast<int>(threadIdx.x) % 256, 1 + sub};
  TopkShared* sh_all = reinterpret_cast<TopkShared*>(cl_smem + kSubBlocks * kScratch);
  uint32_t* cl_keys = reinterpret_cast<uint32_t*>(cl_smem + ClusterSmem<D>::kFixed);
  const int h = static_cast<int>(blockIdx.x) / cluster_ctas;
  const int slot = (static_cast<int>(blockIdx.x) % cluster_ctas) * kSubBlocks + sub;
  const int n_slots = cluster_ctas * kSubBlocks;
  const int n_chunks = (cand_geom<MIXED>(a).nc + kScoreBlocksPerCta - 1) / kScoreBlocksPerCta;
  // (one list per head: the launcher sends per-tile selections to the grid-barrier form)
  // The key sums of this block's first score item are requested first, ahead of the wait for the
  // kernel before this one: that kernel (the query tile sums) writes none of them, and it has itself
  // waited for everything before it, so they are final when any CTA of this grid runs.
  ScoreOperands<D, MIXED> op;
  if (slot < n_chunks) scores_load<D, MIXED>(blk, a, slot, h, op);
  // A CTA's shared memory may be written by its peers only once it runs: every CTA says so here and
  // checks, before its first such write, that all of the cluster have (the two halves of one
  // cluster barrier; by then nobody waits).
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  // launched as a programmatic dependent: the kernel before this one is complete from here on
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // The head's mean query, once per CTA: all 768 threads add up the tile sums (a column's partials
  // split over 768 / D ways, every load of a thread in flight at once, fp64, fixed order), then one
  // thread per column adds the ways.  The three sub-blocks share the result.
  double* qmean = reinterpret_cast<double*>(cl_smem);  // [D], then the per-way partial sums [WAYS][D]
  {
    constexpr int WAYS = 256 * kSubBlocks / D;
    constexpr int kInFlight = 8;
    const int tid = static_cast<int>(threadIdx.x), col = tid % D, way = tid / D;
    const int n_tiles = (a.n_q + kTileM - 1) / kTileM;
    double sum = 0.0;
    for (int t0 = way; t0 < n_tiles; t0 += kInFlight * WAYS) {
      float v[kInFlight];
#pragma unroll
      for (int i = 0; i < kInFlight; ++i)
        v[i] = (t0 + i * WAYS < n_tiles) ? __ldcg(&a.qpart[(static_cast<size_t>(t0 + i * WAYS) * a.H + h) * D + col]) : 0.f;
#pragma unroll
      for (int i = 0; i < kInFlight; ++i) sum += static_cast<double>(v[i]);
    }
    qmean[D + way * D + col] = sum;
    __syncthreads();
    if (tid < D) {
      double t = 0.0;
#pragma unroll
      for (int w = 0; w < WAYS; ++w) t += qmean[D + w * D + tid];
      qmean[tid] = t / static_cast<double>(a.n_q) * static_cast<double>(a.scale);
    }
    __syncthreads();
  }
  // the budgets are asked for now by the block that will need them, far ahead of their use
  int budget = 0, intra_budget = -1;
  if (slot == 0) {
    budget = a.budgets[h];
    if (MIXED && a.intra_budgets) intra_budget = a.intra_budgets[h];
  }
  // the score keys go straight into the key array of the cluster's first CTA (distributed shared
  // memory), where the lists are extracted: no trip through global memory between the two stages
  uint32_t keys_addr;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(keys_addr) : "r"(static_cast<uint32_t>(__cvta_generic_to_shared(cl_keys))), "r"(0u));
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");  // every CTA of the cluster is running
  for (int chunk = slot; chunk < n_chunks; chunk += n_slots)
    scores_item<D, MIXED>(blk, a, chunk, 0, h, qmean, op, false, chunk == slot, keys_addr);
  cluster_sync_all();  // the score keys of the head are complete and visible to its first CTA
  // the kernel behind this one may take the places of the CTAs that leave now
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (slot == 0) topk_item<MIXED>(blk, a, 0, h, cl_keys, sh_all, budget, intra_budget, true);
}

// ---------------------------------------------------------------------------------------
// Head-adaptive selection (Appendix "Sparse Branch"): block weights p = softmax of the pooled
// scores over the candidates, sorted in descending order; Gini coefficient of the sorted weights
// per (head, group); tau_h = tau_min + mean_g(Gini) (tau_max - tau_min); the selection is the
// shortest sorted prefix whose mass reaches tau_h.  Two kernels after the score kernel:
//   adaptive_sort_kernel  one CTA per (group, head): bitonic sort of (score, block) pairs,
//                         fp64 softmax numerators in sorted order, Gini of the group
//   adaptive_pick_kernel  one CTA per (group, head): threshold of the head, prefix length by an
//                         fp64 scan, ascending list of the chosen blocks
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float key_to_float(uint32_t k) {
  const uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
  return __uint_as_float(u);
}

__device__ __forceinline__ double block_sum_f64(double v, double* scratch /*[256]*/) {
  scratch[threadIdx.x] = v;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (static_cast<int>(threadIdx.x) < o) scratch[threadIdx.x] += scratch[threadIdx.x + o];
    __syncthreads();
  }
  const double r = scratch[0];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(256) adaptive_sort_kernel(SelectArgs a, AdaptiveArgs ad) {
  extern __shared__ unsigned long long skeys[];  // [np2]
  __shared__ double scratch[256];
  const int g = blockIdx.x, h = blockIdx.y;
  const int64_t nblk = (a.n_tokens + kBlock - 1) / kBlock;
  const int gtok = a.group_tokens > 0 ? a.group_tokens : a.n_q;
  const int q_hi = min(a.n_q, g * gtok + gtok);
  const int64_t p_last = a.q_pos0 + q_hi - 1;
  int64_t ncand64 = nblk;
  if (a.causal) ncand64 = max64(0, min64(nblk, p_last / kBlock + (p_last >= 0 ? 1 : 0)));
  const int ncand = static_cast<int>(ncand64);
  int np2 = 1;
  while (np2 < ncand) np2 <<= 1;
  const uint32_t* gkeys = a.keys + (static_cast<size_t>(h) * a.n_groups + g) * a.max_pages;
  for (int i = threadIdx.x; i < np2; i += 256)
    skeys[i] = i < ncand ? ((static_cast<unsigned long long>(gkeys[i]) << 32) | (0xffffffffu - static_cast<uint32_t>(i)))
                         : 0ull;  // padding sorts last
  __syncthreads();
  // bitonic sort, descending: larger score first, equal scores -> lower block index first
  for (int k = 2; k <= np2; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = threadIdx.x; i < np2; i += 256) {
        const int ixj = i ^ j;
        if (ixj > i) {
          const unsigned long long x = skeys[i], y = skeys[ixj];
          const bool desc = (i & k) == 0;
          if (desc ? (x < y) : (x > y)) {
            skeys[i] = y;
            skeys[ixj] = x;
          }
        }
      }
      __syncthreads();
    }
  }
  const size_t base = (static_cast<size_t>(h) * a.n_groups + g) * a.max_pages;
  const double smax = ncand > 0 ? static_cast<double>(key_to_float(static_cast<uint32_t>(skeys[0] >> 32))) : 0.0;
  double esum = 0.0, gsum = 0.0;
  for (int m = threadIdx.x; m < ncand; m += 256) {
    const unsigned long long kv = skeys[m];
    const double sc = static_cast<double>(key_to_float(static_cast<uint32_t>(kv >> 32)));
    const double e = exp(sc - smax);
    ad.sorted_w[base + m] = e;
    ad.sorted_idx[base + m] = static_cast<int32_t>(0xffffffffu - static_cast<uint32_t>(kv & 0xffffffffu));
    esum += e;
    gsum += static_cast<double>(ncand - 2 * (m + 1) + 1) * e;
  }
  esum = block_sum_f64(esum, scratch);
  gsum = block_sum_f64(gsum, scratch);
  if (threadIdx.x == 0) {
    ad.wsum[static_cast<size_t>(h) * a.n_groups + g] = esum;
    ad.gini_part[static_cast<size_t>(h) * a.n_groups + g] =
        (ncand > 0 && esum > 0.0) ? gsum / (esum * static_cast<double>(ncand)) : 0.0;
  }
}

__global__ void __launch_bounds__(256) adaptive_pick_kernel(SelectArgs a, AdaptiveArgs ad) {
  extern __shared__ unsigned char flags[];  // [ncand] 1 = selected
  __shared__ double scratch[256];
  __shared__ int warp_sums[8];
  __shared__ int sh_k;
  const int g = blockIdx.x, h = blockIdx.y;
  const int64_t nblk = (a.n_tokens + kBlock - 1) / kBlock;
  const int gtok = a.group_tokens > 0 ? a.group_tokens : a.n_q;
  const int q_hi = min(a.n_q, g * gtok + gtok);
  const int64_t p_last = a.q_pos0 + q_hi - 1;
  int64_t ncand64 = nblk;
  if (a.causal) ncand64 = max64(0, min64(nblk, p_last / kBlock + (p_last >= 0 ? 1 : 0)));
  const int ncand = static_cast<int>(ncand64);
  // threshold of the head: mean Gini over the groups, in group order
  double gmean = 0.0;
  for (int gg = 0; gg < a.n_groups; ++gg) gmean += ad.gini_part[static_cast<size_t>(h) * a.n_groups + gg];
  gmean /= static_cast<double>(a.n_groups);
  const double tau = static_cast<double>(ad.tau_min) + gmean * (static_cast<double>(ad.tau_max) - static_cast<double>(ad.tau_min));
  if (threadIdx.x == 0 && g == 0 && ad.gini_out) {
    ad.gini_out[h] = static_cast<float>(gmean);
    ad.gini_out[a.H + h] = static_cast<float>(tau);
  }
  const size_t base = (static_cast<size_t>(h) * a.n_groups + g) * a.max_pages;
  const double target = tau * ad.wsum[static_cast<size_t>(h) * a.n_groups + g];  // mass to reach
  // prefix length: thread t owns the sorted positions [t*per, t*per + per)
  const int per = (ncand + 255) / 256;
  const int lo = min(ncand, static_cast<int>(threadIdx.x) * per), hi = min(ncand, lo + per);
  double local = 0.0;
  for (int m = lo; m < hi; ++m) local += ad.sorted_w[base + m];
  // exclusive prefix of the per-thread sums, in thread order
  scratch[threadIdx.x] = local;
  __syncthreads();
  double before = 0.0;
  for (int t = 0; t < static_cast<int>(threadIdx.x); ++t) before += scratch[t];
  if (threadIdx.x == 0) sh_k = ncand;  // mass never reached (rounding at tau ~ 1): keep everything
  __syncthreads();
  {
    double cum = before;
    for (int m = lo; m < hi; ++m) {
      cum += ad.sorted_w[base + m];
      if (cum >= target) {
        atomicMin(&sh_k, m + 1);
        break;
      }
    }
  }
  for (int i = threadIdx.x; i < ncand; i += 256) flags[i] = 0;
  __syncthreads();
  const int kk = sh_k;
  for (int m = threadIdx.x; m < kk; m += 256) flags[ad.sorted_idx[base + m]] = 1;
  __syncthreads();
  // ascending compaction of the flagged blocks
  int my_sel = 0;
  for (int b = lo; b < hi; ++b) my_sel += flags[b];
  int total = 0;
  int pos = block_exclusive_scan(Blk{static_cast<int>(threadIdx.x), 0}, my_sel, warp_sums, &total);
  int32_t* out = a.sel_idx + (static_cast<size_t>(h) * a.n_groups + g) * a.kcap;
  for (int b = lo; b < hi; ++b) {
    if (flags[b]) {
      if (pos < a.kcap) out[pos] = b;
      ++pos;
    }
  }
  if (threadIdx.x == 0) {
    a.sel_cnt[static_cast<size_t>(h) * a.n_groups + g] = min(total, a.kcap);
    if (total > a.kcap) atomicCAS(a.status, 0, kDevBounds);
  }
}

cudaError_t launch_select_adaptive(const SelectArgs& a, const AdaptiveArgs& ad, cudaStream_t st) {
  const int n_tiles = (a.n_q + kTileM - 1) / kTileM;
  dim3 g1(n_tiles, a.H);
  if (a.D == 128)
    qsum_partial_kernel<128><<<g1, 256, 0, st>>>(a);
  else
    qsum_partial_kernel<64><<<g1, 256, 0, st>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int64_t nblk = (a.n_tokens + kBlock - 1) / kBlock;
  if (nblk > 0) {
    dim3 g2(static_cast<unsigned>((nblk + kScoreBlocksPerCta - 1) / kScoreBlocksPerCta), a.n_groups, a.H);
    if (a.D == 128)
      block_scores_kernel<128, false><<<g2, 256, 0, st>>>(a);
    else
      block_scores_kernel<64, false><<<g2, 256, 0, st>>>(a);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  int np2 = 1;
  while (np2 < nblk) np2 <<= 1;
  const size_t smem_sort = static_cast<size_t>(np2) * 8;
  if (smem_sort > 40 * 1024)
    cudaFuncSetAttribute(adaptive_sort_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         static_cast<int>(smem_sort));
  dim3 g3(a.n_groups, a.H);
  adaptive_sort_kernel<<<g3, 256, smem_sort, st>>>(a, ad);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  adaptive_pick_kernel<<<g3, 256, static_cast<size_t>(nblk > 0 ? nblk : 1), st>>>(a, ad);
  return cudaGetLastError();
}

namespace {
// cooperative launch support and SM count of the current device (queried once per device)
bool coop_info(int* nsm) {
  static int cached_dev = -1, cached_coop = 0, cached_sm = 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  if (dev != cached_dev) {
    cudaDeviceGetAttribute(&cached_coop, cudaDevAttrCooperativeLaunch, dev);
    cudaDeviceGetAttribute(&cached_sm, cudaDevAttrMultiProcessorCount, dev);
    cached_dev = dev;
  }
  *nsm = cached_sm;
  return cached_coop != 0 && cached_sm > 0;
}
}  // namespace


cudaError_t launch_qsum(const SelectArgs& a, cudaStream_t st) {
  const int n_tiles = (a.n_q + kTileM - 1) / kTileM;
  dim3 g1(n_tiles, a.H);
  if (a.D == 128)
    qsum_partial_kernel<128><<<g1, 256, 0, st>>>(a);
  else
    qsum_partial_kernel<64><<<g1, 256, 0, st>>>(a);
  return cudaGetLastError();
}

namespace {
// Cluster size (8 CTAs, the portable maximum) if the cluster form can be launched on this device for
// the given instance and shared-memory size, else 0.
int cluster_size_for(const void* fn, size_t smem, int threads) {
  const int cs = 8;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(cs);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, fn, &cfg) == cudaSuccess && n >= 1) return cs;
  cudaGetLastError();
  return 0;
}

// One launch as a programmatic dependent of the kernel before it on the stream.
cudaError_t launch_pdl(const void* fn, dim3 grid, dim3 block, size_t smem, void** params, cudaStream_t st,
                       int cluster = 0, bool cooperative = false) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[3];
  int n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n++].val.programmaticStreamSerializationAllowed = 1;
  if (cluster > 0) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[n].val.clusterDim.y = 1;
    attr[n++].val.clusterDim.z = 1;
  }
  if (cooperative) {
    attr[n].id = cudaLaunchAttributeCooperative;
    attr[n++].val.cooperative = 1;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelExC(&cfg, fn, params);
}
}  // namespace

// Three forms, all programmatic dependents of the kernel before them:
//   cluster form        query tile sums as a kernel of their own (they read the whole chunk and want
//                       every SM), then one cluster of 8 CTAs per head for scores and lists, with one
//                       hardware cluster barrier between them -- the default for one list per head while
//                       a head has at most kClusterMaxChunks score items (6144 blocks; measured against
//                       the grid-barrier form: 17.1 against 20.0 us at 2194 blocks, 24.8 against 25.1 us
//                       at 4388)
//   grid-barrier form   one cooperative launch over all SMs with two device barriers -- histories
//                       beyond that, one list per query tile (37 x H lists want more than 24 blocks
//                       of threads per head), and on request
//   three launches      for devices without cooperative launch and for callers without a barrier word
constexpr int kClusterMaxChunks = 192;

cudaError_t launch_select(const SelectArgs& a, cudaStream_t st) {
  int nsm = 0;
  const bool mixed = a.inter_pages > 1 || a.intra_first_page1 > 0 || a.kv_pages != nullptr;
  const int64_t nblk_all = (a.n_tokens + kBlock - 1) / kBlock;
  const int n_tiles = (a.n_q + kTileM - 1) / kTileM;
  SelectArgs aa = a;
  void* p_args[1] = {&aa};
  const void* f_qsum = a.D == 128 ? reinterpret_cast<const void*>(qsum_partial_kernel<128>)
                                  : reinterpret_cast<const void*>(qsum_partial_kernel<64>);
  // candidates per head (coarse candidates make fewer; an upper bound is enough to choose the form)
  const int64_t n_chunks_max = (nblk_all + kScoreBlocksPerCta - 1) / kScoreBlocksPerCta;
  if (a.use_clusters && a.n_groups == 1 && n_chunks_max <= kClusterMaxChunks) {
    const size_t key_bytes = static_cast<size_t>(nblk_all > 0 ? nblk_all : 1) * sizeof(uint32_t);
    const size_t fixed = a.D == 128 ? ClusterSmem<128>::kFixed : ClusterSmem<64>::kFixed;
    const size_t smem = fixed + key_bytes;
    const void* fn = a.D == 128 ? (mixed ? reinterpret_cast<const void*>(select_cluster_kernel<128, true>)
                                         : reinterpret_cast<const void*>(select_cluster_kernel<128, false>))
                                : (mixed ? reinterpret_cast<const void*>(select_cluster_kernel<64, true>)
                                         : reinterpret_cast<const void*>(select_cluster_kernel<64, false>));
    // the cluster size is looked up once per instance, for the largest shared-memory size the form
    // is used with (a cluster that fits with that fits with less)
    constexpr size_t kMaxSmem = 96 * 1024;
    static int cached_cs[2][2] = {{-1, -1}, {-1, -1}};  // [D == 128][mixed]
    int& cs = cached_cs[a.D == 128][mixed];
    bool ok = smem <= kMaxSmem;
    if (ok && cs < 0) {
      ok = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kMaxSmem)) == cudaSuccess;
      cs = ok ? cluster_size_for(fn, kMaxSmem, 256 * kSubBlocks) : 0;
    }
    if (ok && cs > 0) {
      cudaError_t e1 = launch_pdl(f_qsum, dim3(n_tiles, a.H), dim3(256), 0, p_args, st);
      if (e1 != cudaSuccess) return e1;
      int cs_arg = cs;
      void* params[2] = {&aa, &cs_arg};
      return launch_pdl(fn, dim3(static_cast<unsigned>(cs * a.H)), dim3(256 * kSubBlocks), smem, params, st, cs);
    }
    cudaGetLastError();  // no cluster of that shape on this device: the forms below
  }
  if (a.barrier && coop_info(&nsm)) {
    // one cooperative launch for all three stages
    const size_t smem_keys = static_cast<size_t>(nblk_all > 0 ? nblk_all : 1) * sizeof(uint32_t);
    const void* fn = a.D == 128 ? (mixed ? reinterpret_cast<const void*>(select_fused_kernel<128, true>)
                                         : reinterpret_cast<const void*>(select_fused_kernel<128, false>))
                                : (mixed ? reinterpret_cast<const void*>(select_fused_kernel<64, true>)
                                         : reinterpret_cast<const void*>(select_fused_kernel<64, false>));
    if (smem_keys > 24 * 1024)
      cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_keys));
    // 256 threads, at most 80 registers and under 12 KB of shared memory per CTA plus the keys:
    // three CTAs per SM are co-resident while the keys stay below 48 KB
    int per_sm = 3;
    if (smem_keys > 48 * 1024) {
      int occ = 0;
      if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, fn, 256, smem_keys) != cudaSuccess || occ < 1) occ = 1;
      per_sm = occ < 3 ? occ : 3;
    }
    // cooperative: all CTAs co-resident, they meet at two grid barriers
    return launch_pdl(fn, dim3(static_cast<unsigned>(nsm * per_sm)), dim3(256), smem_keys, p_args, st, 0, true);
  }
  // three launches, each a programmatic dependent of the one before
  cudaError_t e = launch_pdl(f_qsum, dim3(n_tiles, a.H), dim3(256), 0, p_args, st);
  if (e != cudaSuccess) return e;
  if (nblk_all > 0) {
    dim3 g2(static_cast<unsigned>(n_chunks_max), a.n_groups, a.H);
    const void* f2 = a.D == 128 ? (mixed ? reinterpret_cast<const void*>(block_scores_kernel<128, true>)
                                         : reinterpret_cast<const void*>(block_scores_kernel<128, false>))
                                : (mixed ? reinterpret_cast<const void*>(block_scores_kernel<64, true>)
                                         : reinterpret_cast<const void*>(block_scores_kernel<64, false>));
    e = launch_pdl(f2, g2, dim3(256), 0, p_args, st);
    if (e != cudaSuccess) return e;
  }
  const size_t smem = static_cast<size_t>(nblk_all > 0 ? nblk_all : 1) * sizeof(uint32_t);
  const void* f3 = mixed ? reinterpret_cast<const void*>(topk_kernel<true>) : reinterpret_cast<const void*>(topk_kernel<false>);
  if (smem > 40 * 1024) cudaFuncSetAttribute(f3, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  return launch_pdl(f3, dim3(a.n_groups, a.H), dim3(256), smem, p_args, st);
}

}  // namespace hsa

// ---------------------------------------------------------------------------------------
// Allocation-free variant of the block selection (no context, no caller workspace).
// Its scratch -- the per-tile query partial sums and the score keys -- lives in a fixed array
// that is part of the library image.  Every GPU that loads the library carries that array
// until the process exits, and all calls share it.
// ---------------------------------------------------------------------------------------
namespace {

constexpr size_t kNoAllocQpartFloats = 64 * 2048;   // up to 64 query tiles x (heads * dim <= 2048)
constexpr size_t kNoAllocKeys = 128 * 1024;         // heads * blocks <= 131072
constexpr size_t kNoAllocScratchBytes = 256 + kNoAllocQpartFloats * 4 + kNoAllocKeys * 4;
static __device__ __align__(256) unsigned char g_select_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_dev_ptr[kMaxDevices] = {nullptr};

// The array's name is only a host-side handle; the device address has to be looked up, once per
// device and with that device current.
int scratch_pointer(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return HSA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_dev_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_select_scratch) != cudaSuccess || ptr == nullptr) return HSA_ERR_CUDA;
    g_scratch_dev_ptr[dev] = ptr;
  }
  *out = g_scratch_dev_ptr[dev];
  return HSA_OK;
}

}  // namespace

extern "C" int hsa_select_blocks_noalloc(const void* q, int32_t n_q, int64_t tok_stride,
                                         int64_t head_stride, int32_t num_heads, int32_t head_dim,
                                         const float* ksum_dev, int32_t ksum_head_stride_blocks,
                                         int64_t n_tokens, int64_t q_pos0, int32_t causal,
                                         float softmax_scale, const int32_t* budgets_dev,
                                         int32_t max_topk, int32_t* sel_idx_dev, int32_t* sel_cnt_dev,
                                         int32_t* status_dev, void* stream) {
  using namespace hsa;
  if (!q || !ksum_dev || !budgets_dev || !sel_idx_dev || !sel_cnt_dev) return HSA_ERR_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return HSA_ERR_INVALID_ARG;
  if (num_heads < 1 || n_q < 1 || max_topk < 1 || n_tokens < 0) return HSA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) % 16) != 0 || tok_stride < head_dim || head_stride < head_dim ||
      (tok_stride % 8) != 0 || (head_stride % 8) != 0)
    return HSA_ERR_INVALID_ARG;
  const int64_t nblk = (n_tokens + kBlock - 1) / kBlock;
  if (ksum_head_stride_blocks < nblk) return HSA_ERR_INVALID_ARG;
  // fixed scratch: refuse anything that does not fit
  const int64_t n_tiles = (static_cast<int64_t>(n_q) + kTileM - 1) / kTileM;
  if (n_tiles * num_heads * head_dim > static_cast<int64_t>(kNoAllocQpartFloats) ||
      static_cast<int64_t>(num_heads) * ksum_head_stride_blocks > static_cast<int64_t>(kNoAllocKeys) ||
      nblk * 4 > 200 * 1024)
    return HSA_ERR_OUT_OF_PAGES;
  void* base = nullptr;
  const int rc = scratch_pointer(&base);
  if (rc != HSA_OK) return rc;
  unsigned char* sc = static_cast<unsigned char*>(base);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the first 256 bytes hold a status word for callers that pass none: it has to start at zero
  if (!status_dev && cudaMemsetAsync(sc, 0, 256, st) != cudaSuccess) return HSA_ERR_CUDA;
  SelectArgs a{};
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.n_q = n_q;
  a.tok_stride = tok_stride;
  a.head_stride = head_stride;
  a.q_pos0 = q_pos0;
  a.causal = causal != 0;
  a.n_tokens = n_tokens;
  a.H = num_heads;
  a.D = head_dim;
  a.max_pages = ksum_head_stride_blocks;
  a.ksum = ksum_dev;
  a.budgets = budgets_dev;
  a.group_tokens = 0;
  a.n_groups = 1;
  a.scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(head_dim));
  a.qpart = reinterpret_cast<float*>(sc + 256);
  a.keys = reinterpret_cast<uint32_t*>(sc + 256 + kNoAllocQpartFloats * 4);
  a.sel_idx = sel_idx_dev;
  a.sel_cnt = sel_cnt_dev;
  a.kcap = max_topk;
  a.status = status_dev ? status_dev : reinterpret_cast<int32_t*>(sc);
  // (no grid-barrier counter: this entry point runs the three stages as three launches)
  return launch_select(a, st) == cudaSuccess ? HSA_OK : HSA_ERR_CUDA;
}
