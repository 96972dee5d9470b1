/*
 * hsa.h -- C ABI of the B200-native Hybrid Sparse Attention (HSA) forward path.
 *
 * One context (hsa_ctx) is one attention layer of one sequence (batch 1): a
 * paged KV pool resident in HBM (the device tier of the Hierarchical KV Cache,
 * Section 3.2), the per-block key sums used for block scoring, and the running
 * state of the linear branch.  Per query chunk the caller does
 *
 *     hsa_append_kv      (new K/V of the chunk -> pool pages, key sums, state)
 *     hsa_select_blocks  (pooled scores + per-head top-k, indices stay on device)
 *     hsa_forward        (block-sparse softmax branch + linear branch + gated merge)
 *
 * Conventions that hold for every entry point
 *   - "device" pointers are CUDA device addresses owned by the caller (allocated
 *     with any allocator, e.g. torch); "host" pointers are ordinary host memory.
 *     The library never allocates or frees device memory; a context owns only
 *     host-side bookkeeping.  The caller frees its buffers after hsa_destroy.
 *   - q / k / v / out are bf16 tensors indexed [token][head][dim] with explicit
 *     token and head strides given in ELEMENTS; the dim stride is 1.  Base
 *     addresses and byte strides must be multiples of 16.
 *   - Every call only enqueues work on the given CUDA stream (a cudaStream_t
 *     passed as void*; NULL = default stream) and returns; nothing synchronises
 *     except hsa_device_status.  A context is not thread-safe.
 *   - Return value: HSA_OK (0) or a negative hsa_status.  Device-side problems
 *     (a bounded wait that ran out, an out-of-range block index) never trap:
 *     the kernel records a code in a status word that hsa_device_status reads.
 *   - History tokens form one continuous stream; block b holds tokens
 *     [64 b, 64 b + 64); only the last block may be partial.  Query i of a chunk
 *     sits at absolute position q_pos0 + i.  With causal != 0 key j is visible
 *     to query i iff j <= q_pos0 + i (mask M of the attention definition,
 *     Appendix A.1, Eq. 6).
 */
#ifndef HSA_H_
#define HSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HSA_PAGE_TOKENS 64

typedef enum {
  HSA_OK = 0,
  HSA_ERR_INVALID_ARG = -1,    /* null / misaligned pointer, size out of the configured range   */
  HSA_ERR_OUT_OF_PAGES = -2,   /* append would exceed max_pages                                 */
  HSA_ERR_UNSUPPORTED = -3,    /* valid request this build does not implement                   */
  HSA_ERR_CUDA = -4,           /* a CUDA runtime / driver call failed (see hsa_last_cuda_error)  */
  HSA_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait expired (status word)              */
  HSA_ERR_DEVICE_BOUNDS = -6   /* a device-side index was out of range and was skipped          */
} hsa_status;

/* lin_mode */
#define HSA_LIN_NONE 0
#define HSA_LIN_STATE 1      /* running state S = sum phi(k)^T v, z = sum phi(k); phi: feature_map */
#define HSA_LIN_LINFORMER 2  /* Section 3.3 "Linear branch" (Eq. 3) and Appendix G: per segment of
                                lin_seg_tokens tokens K~ = E_K^T K, V~ = E_V^T V (lin_rank rows each),
                                concatenated; O_lin = Softmax(Q K~^T / sqrt(d)) V~.  head_dim 128 only */

/* feature_map of the running-state linear branch (the paper defines none for this form):
 * phi(x) = elu(x) + 1, the default, or phi(x) = max(x, 0).  With relu a query can have weight zero
 * on every key, so that form divides by (phi(q) . z + 1e-6). */
#define HSA_PHI_ELU1 0
#define HSA_PHI_RELU 1

/* hsa_config.flags: reserve workspace for causal forwards with the linear branch on */
#define HSA_CFG_CAUSAL 1u
/* hsa_config.flags: reserve workspace for hsa_select_blocks_adaptive (needs max_pages <= 8192) */
#define HSA_CFG_ADAPTIVE 2u
/* hsa_config.flags: run the selection kernel in its grid-barrier form (one cooperative launch whose
 * CTAs meet at two device-wide barriers in global memory) instead of the default form, in which the
 * CTAs of a head form a thread-block cluster and meet at hardware cluster barriers.  The library
 * falls back to the grid-barrier form by itself where clusters of 8 CTAs cannot be launched. */
#define HSA_CFG_GRID_BARRIER_SELECT 4u

/* hsa_forward flags: the paper's "linear only" / "sparse only" ablation modes (Table 4) */
#define HSA_FWD_NO_LINEAR 1u
#define HSA_FWD_NO_SPARSE 2u

typedef struct hsa_ctx hsa_ctx;

typedef struct {
  int32_t num_heads;      /* H >= 1                                                            */
  int32_t head_dim;       /* 64 or 128                                                         */
  int32_t page_tokens;    /* must be HSA_PAGE_TOKENS                                           */
  int32_t max_pages;      /* pool capacity in pages (= KV blocks)                              */
  int32_t max_q_tokens;   /* largest query chunk / appended chunk                              */
  int32_t max_topk;       /* row capacity of sel_idx (blocks per head and query group)         */
  int32_t lin_mode;       /* HSA_LIN_*                                                         */
  int32_t gate_act;       /* 0: gates used as given; 1: sigmoid(gate) (Section 3.3, Eq. 5)     */
  float softmax_scale;    /* 0 -> 1/sqrt(head_dim)                                             */
  uint32_t flags;         /* HSA_CFG_* bits                                                    */
  int32_t lin_rank;       /* HSA_LIN_LINFORMER: projection rank r, a multiple of 64, 64..2048 (else 0) */
  int32_t lin_seg_tokens; /* HSA_LIN_LINFORMER: segment length L; every append must be exactly L      */
  int32_t split_blocks;   /* a (query tile, head) with more selected blocks than this is split over
                             several CTAs whose partial results the last one to finish merges
                             (0 -> 256; only matters when max_topk exceeds it)                     */
  int32_t feature_map;    /* HSA_LIN_STATE: HSA_PHI_ELU1 (0) or HSA_PHI_RELU                           */
} hsa_config;

typedef struct {
  size_t k_pool;     /* bytes: [max_pages][H][64][d] bf16                                      */
  size_t v_pool;     /* same                                                                   */
  size_t state;      /* linear-branch state + per-block key sums                               */
  size_t workspace;  /* page table copy, partial sums, status word                             */
  size_t kc_pool;    /* HSA_LIN_LINFORMER: compressed keys, [segments * r / 64][H][64][d] bf16, else 0  */
  size_t vc_pool;    /* same for the compressed values                                         */
} hsa_sizes;

typedef struct {
  void* k_pool;     /* device, 256-byte aligned                                                */
  void* v_pool;     /* device, 256-byte aligned                                                */
  void* state;      /* device, 256-byte aligned; zero-filled by hsa_create (synchronously)     */
  void* workspace;  /* device, 256-byte aligned                                                */
  void* kc_pool;    /* HSA_LIN_LINFORMER only (else NULL): device, 256-byte aligned            */
  void* vc_pool;
  const void* e_k;  /* HSA_LIN_LINFORMER only: device bf16 [H][lin_seg_tokens][lin_rank], 16-byte aligned */
  const void* e_v;
} hsa_buffers;

/* Bytes the caller must allocate for a configuration.  Host only, no CUDA call. */
int hsa_query_sizes(const hsa_config* cfg, hsa_sizes* out);

/* Creates a context over caller-owned device buffers of at least hsa_query_sizes bytes.
 * page_alloc_order_host: host int32[max_pages], a permutation of 0..max_pages-1 giving the
 * physical page assigned to the b-th block of the history (NULL = identity).  The page table
 * is copied to the workspace and the state is cleared, synchronously. */
int hsa_create(hsa_ctx** out, const hsa_config* cfg, const hsa_buffers* bufs,
               const int32_t* page_alloc_order_host);

/* Appends n_tokens (1..max_q_tokens) new history tokens:
 * writes K/V rows into pool pages through the page table (continuing a partial tail
 * page), updates the per-(head, block) key sums used by the pooled block scores
 * (Section 3.3 "Sparse branch"; Section 3.2 Stage 2 "average key"), and the linear state
 * S[h] += sum_j phi(k_j)^T v_j, z[h] += sum_j phi(k_j) (fp32), keeping the previous state
 * for causal forwards.   k, v: device bf16 [n_tokens][H][d] with the given strides. */
int hsa_append_kv(hsa_ctx* ctx, const void* k, const void* v, int32_t n_tokens,
                  int64_t tok_stride, int64_t head_stride, void* stream);

/* Pooled block scores s[h,g,b] = mean_q(group g) . mean_k(block b) * scale
 * (Section 3.2 Stage 2 score form) and, per (head, group), the min(budget, candidates)
 * highest-scoring candidate blocks; exact ties go to the lower block index.
 *   budgets_dev      device int32[H]; < 0 or >= candidates selects every candidate.
 *   q_group_tokens   0 = one selection for the whole chunk; otherwise a multiple of 128.
 *   sel_idx_dev      device int32[H][n_groups][max_topk], ascending block ids (output).
 *   sel_cnt_dev      device int32[H][n_groups] (output).
 * Candidates: blocks with at least one token and, if causal, first token <= last query
 * position of the group.  Counts are clamped to max_topk (flagged in the status word).
 * The work is enqueued as one or two kernels (see HSA_CFG_GRID_BARRIER_SELECT); the lists are the
 * same bit for bit either way. */
int hsa_select_blocks(hsa_ctx* ctx, const void* q, int32_t n_q, int64_t tok_stride,
                      int64_t head_stride, int64_t q_pos0, int32_t causal,
                      const int32_t* budgets_dev, int32_t q_group_tokens,
                      int32_t* sel_idx_dev, int32_t* sel_cnt_dev, void* stream);

/* Selection with the two sparse granularities of Section 3.3 ("Inter- and intra-chunk sparse
 * granularity"): history before the current chunk is scored and selected in coarse blocks of
 * inter_block_pages pages (2 = the paper's B_inter = 128 tokens), the current chunk's own tokens in
 * single pages (B_intra = 64); both kinds come out as one ascending list of 64-token pages, so the
 * forward kernel is the same.
 *   inter_block_pages   1 or 2 (0 = 1).  A coarse block is scored by the mean key over all of its
 *                       tokens; selecting it selects its pages.  budgets_dev counts coarse blocks.
 *   intra_first_page    first page of the current chunk (the page that holds its first token), or
 *                       < 0 for no intra-chunk region.  Pages from here on are candidates of their
 *                       own, outside budgets_dev.
 *   intra_budgets_dev   device int32[H] budgets for those pages, or NULL = every one of them
 *                       (the chunk always attends to itself).
 *   kv_pages_dev        device int32[n_kv_pages]: ids of the KV pages kept by hsa_retrieve_kv_pages
 *                       (runs of kv_page_blocks blocks), or NULL for no mask.  An inter-chunk block
 *                       with a page outside them is no candidate at all: the retrieved pages are
 *                       the ones that are resident (Section 3.2, "Active KV construction").  The
 *                       chunk's own pages are never masked.
 * max_topk must hold inter_block_pages * budget + the intra-chunk pages.  opts == NULL is
 * hsa_select_blocks.  Everything else as hsa_select_blocks. */
typedef struct {
  int32_t inter_block_pages;
  int32_t intra_first_page;
  const int32_t* intra_budgets_dev;
  const int32_t* kv_pages_dev;
  int32_t n_kv_pages;
  int32_t kv_page_blocks;
} hsa_select_opts;
int hsa_select_blocks_ex(hsa_ctx* ctx, const void* q, int32_t n_q, int64_t tok_stride,
                         int64_t head_stride, int64_t q_pos0, int32_t causal,
                         const int32_t* budgets_dev, int32_t q_group_tokens,
                         const hsa_select_opts* opts, int32_t* sel_idx_dev, int32_t* sel_cnt_dev,
                         void* stream);

/* Page-level retrieval of the hierarchical KV cache (Section 3.2, Stage 2).  A KV page is a run of
 * kv_page_blocks consecutive 64-token blocks of the history (the paper's page of 8 frames x 1560
 * tokens is 195 blocks).  Its score is alpha_j = Qbar . Kbar_j * scale with the average query of the
 * chunk and the average key of the page, averaged over the heads (the paper is silent on heads: one
 * set of pages serves the whole layer); the top_kp best pages (the paper uses K_p = 4; ties to the
 * lower id) are written in ascending order.
 *   page_ids_dev   device int32[min(top_kp, pages)] (output); pages = ceil(blocks / kv_page_blocks)
 *   scores_dev     device fp32[pages] receiving every alpha_j, or NULL
 *   n_out_host     host int32 receiving min(top_kp, pages) (known without a device read), or NULL
 * The ids feed hsa_select_opts.kv_pages_dev.  HSA_ERR_UNSUPPORTED above 2048 pages. */
int hsa_retrieve_kv_pages(hsa_ctx* ctx, const void* q, int32_t n_q, int64_t tok_stride,
                          int64_t head_stride, int32_t kv_page_blocks, int32_t top_kp,
                          int32_t* page_ids_dev, float* scores_dev, int32_t* n_out_host, void* stream);

/* Tier migration of the hierarchical KV cache (Section 3.2: pages that are not retrieved leave the
 * GPU for host memory and come back on demand).  The K and V tiles of history blocks
 * [first_block, first_block + n_blocks) are copied to / from caller-owned host buffers laid out as
 * [n_blocks][H][64][d] bf16 (pinned memory makes the copies asynchronous), one copy per run of
 * physically adjacent pages, on the given stream.  The context only tracks residency on the host:
 * an evicted block keeps its key sum (it still takes part in scoring) but its tiles must be restored
 * before a forward call selects it -- restrict the selection with kv_pages_dev, or check with
 * hsa_block_resident.  Appending to a block marks it resident.  HSA_ERR_INVALID_ARG outside the
 * history. */
int hsa_evict_blocks(hsa_ctx* ctx, int32_t first_block, int32_t n_blocks, void* host_k, void* host_v,
                     void* stream);
int hsa_restore_blocks(hsa_ctx* ctx, int32_t first_block, int32_t n_blocks, const void* host_k,
                       const void* host_v, void* stream);
int hsa_block_resident(hsa_ctx* ctx, int32_t block, int32_t* resident_out);

/* Head-adaptive selection (Appendix F, Eq. 12-13): instead of a given budget, each (head, group)
 * keeps the shortest prefix of its blocks, sorted by pooled score, whose softmax mass reaches
 *   tau_h = tau_min + G_h (tau_max - tau_min),
 * G_h being the Gini coefficient of the sorted block weights averaged over the head's groups
 * (the paper's best setting is tau_max = 1.00, tau_min = 0.35).  Same candidates, tie rule and
 * output layout as hsa_select_blocks.  gini_tau_out_dev: optional device fp32 [2][H] receiving G_h
 * and tau_h.  Needs HSA_CFG_ADAPTIVE; HSA_ERR_UNSUPPORTED when the history has more than 8192
 * blocks. */
int hsa_select_blocks_adaptive(hsa_ctx* ctx, const void* q, int32_t n_q, int64_t tok_stride,
                               int64_t head_stride, int64_t q_pos0, int32_t causal, float tau_min,
                               float tau_max, int32_t q_group_tokens, int32_t* sel_idx_dev,
                               int32_t* sel_cnt_dev, float* gini_tau_out_dev, void* stream);

/* Block selection for callers that cannot allocate device memory (the paper has no counterpart;
 * this is a convenience of this library).  Some callers run where cudaMalloc is off limits --
 * inside a region being captured into a CUDA graph, in a process whose memory pool is owned by
 * another framework, or in a service that forbids allocation after start-up -- and cannot
 * provide the context's workspace either.  This entry point computes exactly what
 * hsa_select_blocks computes for q_group_tokens = 0 (one selection per head for the whole chunk),
 * needs no context, and keeps its scratch (query partial sums and score keys, about 1 MiB) in a
 * fixed array inside the library: every GPU that loads the library holds that array until the
 * process exits.
 *   ksum_dev                  device fp32 [H][ksum_head_stride_blocks][d]: per-(head, block) key
 *                             sums as hsa_append_kv maintains them (see hsa_state_layout)
 *   status_dev                device int32 status word (zeroed by the caller) that receives
 *                             HSA_ERR_DEVICE_BOUNDS when a list had to be cut at max_topk; with NULL
 *                             the flag goes to a word inside the scratch that no entry point reads,
 *                             i.e. a cut list is then not reported: pass a word when max_topk may
 *                             be smaller than a budget
 * Limits (HSA_ERR_OUT_OF_PAGES beyond them): ceil(n_q/128) * H * d <= 131072,
 * H * ksum_head_stride_blocks <= 131072, ceil(n_tokens/64) <= 51200.
 * It calls no allocator (no cudaMalloc / cudaFree, no library routine that allocates).  The first
 * call on a device looks up the device address of the scratch array (with that device current);
 * make that first call before any stream capture begins.  All calls share the one array, which
 * keeps the previous call's contents: two calls whose kernels may overlap on the GPU (different
 * streams, or different threads) race on it -- serialise them. */
int hsa_select_blocks_noalloc(const void* q, int32_t n_q, int64_t tok_stride, int64_t head_stride,
                              int32_t num_heads, int32_t head_dim, const float* ksum_dev,
                              int32_t ksum_head_stride_blocks, int64_t n_tokens, int64_t q_pos0,
                              int32_t causal, float softmax_scale, const int32_t* budgets_dev,
                              int32_t max_topk, int32_t* sel_idx_dev, int32_t* sel_cnt_dev,
                              int32_t* status_dev, void* stream);

/* out[i,h,:] = w(g_lin) * O_lin + w(g_sp) * O_sp  (Section 3.3, Eq. 5), where
 *   O_sp  = softmax attention of query i over the visible keys of the selected blocks
 *           (Eq. 4 with the block mask; Appendix A.1),
 *   O_lin = phi(q_i) S / (phi(q_i) z) over all visible history (running-state form),
 *   w(g)  = 1 if the gate pointer is NULL, else g or sigmoid(g) per gate_act.
 * A branch with nothing visible contributes 0.  sel_idx_dev / sel_cnt_dev may come from
 * hsa_select_blocks or from the caller (same layout).  Gates: device bf16 with element
 * strides (token, head, dim); dim stride 0 broadcasts one gate per (token, head).
 * causal != 0 with the linear branch on requires HSA_CFG_CAUSAL and the query chunk to be the
 * most recently appended chunk (q_pos0 + n_q == tokens appended so far, n_q == size of the
 * last append), otherwise HSA_ERR_UNSUPPORTED; the sparse branch alone takes any q_pos0.  out: device bf16 [n_q][H][d], strides as q. */
int hsa_forward(hsa_ctx* ctx, const void* q, int32_t n_q, int64_t tok_stride, int64_t head_stride,
                int64_t q_pos0, int32_t causal, const int32_t* sel_idx_dev,
                const int32_t* sel_cnt_dev, int32_t q_group_tokens, const void* g_lin,
                const void* g_sp, int64_t gate_tok_stride, int64_t gate_head_stride,
                int64_t gate_dim_stride, void* out, int64_t out_tok_stride,
                int64_t out_head_stride, uint32_t flags, void* stream);

/* Host-tracked length of the history. */
int hsa_get_info(hsa_ctx* ctx, int64_t* n_tokens, int32_t* n_blocks);

/* Sets the history length back to n_tokens (<= current).
 * Undoing exactly the most recent hsa_append_kv (n_tokens = the length before it, no other rewind in
 * between) needs nothing else: the linear state lives in two slots that take turns, so the state
 * before that append is still there, and the key sum its first block had before the append is kept
 * and reused by the next append from that length.  The same chunk, or another one, can then be
 * appended again (benchmarks replay a step this way; a caller can drop a speculative chunk).
 * Any other rewind keeps the pool's pages but recomputes nothing: the caller must put the state
 * buffer (hsa_state_layout) back to the contents it had at that length. */
int hsa_rewind(hsa_ctx* ctx, int64_t n_tokens);

/* Byte offsets inside the state buffer, for tests and snapshots:
 * S fp32 [H][d][d], z fp32 [H][d] (of the slot that holds the current state: the offsets change with
 * every hsa_append_kv and with an undoing hsa_rewind), key sums fp32 [H][max_pages][d]. */
int hsa_state_layout(hsa_ctx* ctx, size_t* off_S, size_t* off_z, size_t* off_ksum);

/* Synchronises the device, reads and clears the status word: HSA_OK or a DEVICE_* code.
 * After HSA_ERR_DEVICE_TIMEOUT the selection written by the call that timed out has every count
 * set to zero (a forward call on it computes the linear branch alone), and this call also puts
 * the selection kernel's grid barrier back to its initial state, so the next call starts clean. */
int hsa_device_status(hsa_ctx* ctx, int32_t* status_out);

/* Bound, in nanoseconds, of a wait at the grid barrier of the selection kernel (the one place
 * where CTAs wait for each other; default 2e9).  When it runs out the kernel ends, the status word
 * holds HSA_ERR_DEVICE_TIMEOUT and the call's selection is empty.  wait_ns > 0. */
int hsa_set_wait_limit_ns(hsa_ctx* ctx, uint64_t wait_ns);

/* Byte offsets inside the workspace, for tests and monitoring: the int32 status word, and the
 * two uint32 words {arrive count, generation} of the selection kernel's grid barrier, which the
 * kernel updates together as one 8-byte word (off_barrier is 8-byte aligned; the count is zero
 * whenever no selection kernel is running; the generation advances by two per launch of the
 * grid-barrier form). */
int hsa_workspace_layout(hsa_ctx* ctx, size_t* off_status, size_t* off_barrier);

/* Synchronises the device, reads and clears a counter: the number of (query tile, head) work
 * items since the last read whose softmax had to be redone with a running maximum because a
 * later key block outscored the first block of the tile by more than about 2^47 (the normal
 * pass fixes the exponent reference once per tile; results are the same, the redo only costs
 * time).  Informational. */
int hsa_safe_pass_tiles(hsa_ctx* ctx, int64_t* count_out);

/* Last CUDA error code recorded by a failing call on this context (0 if none). */
int hsa_last_cuda_error(hsa_ctx* ctx);

int hsa_destroy(hsa_ctx* ctx);

const char* hsa_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* HSA_H_ */
