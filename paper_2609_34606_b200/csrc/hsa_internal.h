// Internal declarations shared by the C-ABI layer and the kernel launchers.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/hsa.h"

namespace hsa {

constexpr int kBlock = HSA_PAGE_TOKENS;  // tokens per KV block = tokens per page
constexpr int kTileM = 128;              // query rows per work item of the forward kernel
constexpr int kStateSplitMax = 16;       // token-axis splits of the state update (per head)
// z as a [16 x 128] bf16 K-major operand image (128-byte swizzle, two slabs of 64 dims): row 0 holds
// the bf16 rounding of z, row 1 the bf16 rounding of the remainder, rows 2..15 are zero, so that
// phi(Q) times it gives the denominator phi(q).z as the sum of two accumulator columns
constexpr int kZopBytes = 4096;
constexpr int kFwdSplitMax = 16;         // CTAs a long (query tile, head) of the forward kernel is split over

__host__ __device__ inline int64_t min64(int64_t a, int64_t b) { return a < b ? a : b; }
__host__ __device__ inline int64_t max64(int64_t a, int64_t b) { return a > b ? a : b; }

// device status word values (match hsa_status)
constexpr int kDevTimeout = HSA_ERR_DEVICE_TIMEOUT;
constexpr int kDevBounds = HSA_ERR_DEVICE_BOUNDS;

struct AppendArgs {
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  int n_new;
  int64_t tok_stride, head_stride;
  int64_t n0;  // tokens already in the history
  int H, D, max_pages;
  const int32_t* page_table;
  __nv_bfloat16* k_pool;
  __nv_bfloat16* v_pool;
  float* ksum;      // [H][max_pages][D]
  // The running state lives in two slots that take turns: an append reads slot src_slot and writes
  // slot src_slot ^ 1, which becomes the current one; the other keeps the state before the append
  // (what a causal forward over the appended chunk applies, and what undoing the append returns to).
  float* S[2];          // [H][D][D] per slot
  float* z[2];          // [H][D] per slot
  int src_slot;
  __nv_bfloat16* hilo;  // [H][2 slots][2 hi/lo][D][D]: bf16 hi + lo of S, what the forward kernels read
  uint8_t* zop;         // [H][2 slots][kZopBytes]: z as a tensor-core operand (head_dim 128)
  // key sum the (partly filled) first block of this append had before it: saved here when the append
  // reads it from ksum, read from here instead when the append repeats one that was undone
  float* ksum_saved;    // [H][D]
  int tail_from_saved;
  float* spart;         // [H][nsplit][D*D + D] scratch
  int nsplit;
  int lin_state;  // update the linear state?
  int beside_prior;  // SIMT page write: may run beside the kernel launched just before it (see launch_append)
  int relu;       // feature map of the state: 0 elu(x) + 1, 1 max(x, 0)
  int32_t* status;  // device status word
};

struct SelectArgs {
  const __nv_bfloat16* q;
  int n_q;
  int64_t tok_stride, head_stride;
  int64_t q_pos0;
  int causal;
  int64_t n_tokens;
  int H, D, max_pages;
  const float* ksum;
  const int32_t* budgets;
  int group_tokens, n_groups;
  float scale;
  float* qpart;  // [n_tiles][H][D] scratch
  uint32_t* keys;  // [H][n_groups][max_pages] scratch: order-preserving score keys
  int32_t* sel_idx;
  int32_t* sel_cnt;
  int kcap;
  int32_t* status;
  unsigned* barrier;  // grid barrier of the single-launch path: {arrive count, generation}, the count
                      // zero when no launch is in flight (null: three launches)
  unsigned long long wait_ns;  // bound of a wait at that barrier
  int use_clusters;            // 1: one thread-block cluster per head (hardware cluster barriers) where the device allows
  // candidate geometry: pages before the first intra-chunk page are selected in runs of inter_pages pages against
  // budgets[], the pages from it on one by one against intra_budgets[] (null: all of them)
  int inter_pages;           // 0 or 1: every page on its own
  int64_t intra_first_page1;  // first intra-chunk page + 1; 0: no intra-chunk region
  const int32_t* intra_budgets;
  // retrieved KV pages (runs of kv_page_blocks blocks): an inter-chunk candidate with a page outside
  // them is no candidate (null: no mask)
  const int32_t* kv_pages;
  int n_kv_pages, kv_page_blocks;
};

struct RetrieveArgs {
  int n_q, H, D, max_pages;
  int64_t n_tokens;
  const float* qpart;  // [tiles][H][D] query tile sums
  const float* ksum;   // [H][max_pages][D]
  int kv_page_blocks, top_kp;
  float scale;
  uint32_t* keys;      // [pages] scratch
  float* scores_out;   // [pages] or null
  int32_t* page_ids;   // [min(top_kp, pages)] ascending (output)
};

struct FwdParams {
  int n_q, H;
  int64_t n_tokens;
  int64_t q_pos0;
  int causal;
  const int32_t* sel_idx;
  const int32_t* sel_cnt;
  int kcap, n_groups, group_tokens;
  const int32_t* page_table;
  int n_blocks;
  const float* z;       // [H][D] state the linear branch applies
  const uint8_t* zop;   // [H][2 slots][kZopBytes]: the same z as a tensor-core operand
  int state_slot;       // slot the linear branch applies; row of the hi/lo tensor map = ((h*2 + slot)*2 + hl)*D
  const __nv_bfloat16* g_lin;
  const __nv_bfloat16* g_sp;
  int64_t g_ts, g_hs, g_ds;
  int gate_act;
  __nv_bfloat16* out;
  int64_t o_ts, o_hs;
  float scale_log2;  // softmax scale * log2(e)
  uint32_t flags;
  int do_linear, do_sparse;
  const float* lin_num;  // causal intra-chunk partials [n_q][H][D] (or null)
  const float* lin_den;  // [n_q][H]
  const __nv_bfloat16* ext_lin;  // linear-branch output computed elsewhere, [n_q][H][D] (or null)
  // Linformer form inside the kernel: the loop first runs over the lf_pages pages of the compressed
  // pool (page ids through lf_table), with an accumulator and row sums of their own (null: none)
  const int32_t* lf_table;
  int lf_pages;
  int relu;  // feature map of the state form: 0 elu(x) + 1, 1 max(x, 0) with 1e-6 added to the denominator
  // split tiles: a (tile, head) with more than split_blocks selected blocks runs as several CTAs
  // (grid z = max_splits); each dumps its unnormalised O, row sums and exponent references, the last
  // one to take a ticket merges them and writes the output
  int max_splits, split_blocks;
  int n_tiles, remap;    // set by the launcher: query tiles; 1 = one-dimensional grid, longest lists first
  int nsm;               // SMs of the device (the split rule balances the launch over them)
  float* part_o;         // [tiles][H][max_splits][128][D]
  float* part_l;         // [tiles][H][max_splits][128]
  float* part_ref;       // [tiles][H][max_splits][128]
  int32_t* part_ticket;  // [tiles][H], zero between launches
  int32_t* status;
  // L2 look-ahead of the page gather: the pools themselves (null: none)
  const uint8_t* k_pool;
  const uint8_t* v_pool;
};

struct CausalLinArgs {
  const __nv_bfloat16* q;
  int n_q;
  int64_t q_ts, q_hs;
  const __nv_bfloat16* k_pool;
  const __nv_bfloat16* v_pool;
  const int32_t* page_table;
  int64_t q_pos0;   // first query position == first token of the intra-chunk part
  int64_t n_tokens;
  int H, D;
  int relu;  // feature map: 0 elu(x) + 1, 1 max(x, 0)
  float* lin_num;
  float* lin_den;
};

struct LinformerArgs {
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  int64_t tok_stride, head_stride;
  const __nv_bfloat16* e_k;  // [H][seg_tokens][rank]
  const __nv_bfloat16* e_v;
  __nv_bfloat16* kc_pool;    // [compressed pages][H][64][128]
  __nv_bfloat16* vc_pool;
  int32_t* ccnt;             // [H] number of valid compressed pages
  int H, rank, seg_tokens, seg_index;
  int32_t* status;
};

// tensor maps of the fused append kernel: the chunk's K and V ([tokens][H][d], box 64 dims x 1 x 64
// tokens) and the two pools ([rows][d], box 64 x 64), all with the 128-byte swizzle
struct AppendMaps {
  CUtensorMap kin, vin, kpool, vpool;
};
cudaError_t launch_append(const AppendArgs& a, const AppendMaps* maps, cudaStream_t st);
cudaError_t launch_linformer_compress(const LinformerArgs& a, const CUtensorMap& tm_ek, const CUtensorMap& tm_ev,
                                      const CUtensorMap& tm_kin, const CUtensorMap& tm_vin, cudaStream_t st);
cudaError_t linformer_init();
struct AdaptiveArgs {
  double* sorted_w;      // [H][n_groups][max_pages] softmax numerators in sorted order
  int32_t* sorted_idx;   // [H][n_groups][max_pages] block ids in sorted order
  double* gini_part;     // [H][n_groups]
  double* wsum;          // [H][n_groups] sum of the numerators
  float tau_min, tau_max;
  float* gini_out;       // [2][H]: Gini and threshold per head (or null)
};

cudaError_t launch_select(const SelectArgs& a, cudaStream_t st);
cudaError_t launch_qsum(const SelectArgs& a, cudaStream_t st);  // stage 1 alone: query tile sums
cudaError_t launch_retrieve(const RetrieveArgs& a, int n_pages, cudaStream_t st);
cudaError_t launch_select_adaptive(const SelectArgs& a, const AdaptiveArgs& ad, cudaStream_t st);
// tm_kc / tm_vc: maps of the compressed pools, used when p.lf_table is set (else null)
cudaError_t launch_forward(const FwdParams& p, int D, const CUtensorMap& tm_q,
                           const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                           const CUtensorMap& tm_state, const CUtensorMap& tm_out, cudaStream_t st,
                           const CUtensorMap* tm_kc = nullptr, const CUtensorMap* tm_vc = nullptr);
cudaError_t launch_causal_linear(const CausalLinArgs& a, cudaStream_t st);
// linear branch alone (head_dim 128): lean HBM-bound kernel, nsm = SMs of the device
cudaError_t launch_linear_only(const FwdParams& p, int nsm, const CUtensorMap& tm_q, const CUtensorMap& tm_state,
                               const CUtensorMap& tm_out, cudaStream_t st);
cudaError_t linear_only_init();
cudaError_t forward_init();
cudaError_t append_init();  // opt in to the shared-memory size the fused append kernel needs

}  // namespace hsa
