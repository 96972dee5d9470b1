// C-ABI layer: context bookkeeping, argument validation, tensor maps and kernel launches.
// The library owns no device memory; every device buffer comes from the caller.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "hsa_internal.h"

using namespace hsa;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
  // state
  size_t S, z, slot_S, slot_z, hilo, zop, ksum_saved, ksum, state_total;  // S, z: slot 0; slot_*: bytes per slot
  // workspace
  size_t status, page_table, qpart, keys, spart, lin_num, lin_den, ctable, csel, ccnt, olin, ad_w, ad_idx, ad_gini, ad_wsum,
      part_o, part_l, part_ref, part_ticket, ws_total;
  int fwd_splits, split_blocks;
  // Linformer
  size_t n_cpages, cpool;
};

bool config_ok(const hsa_config* c) {
  if (!c) return false;
  if (c->num_heads < 1 || c->num_heads > 1024) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->page_tokens != HSA_PAGE_TOKENS) return false;
  if (c->max_pages < 1 || c->max_q_tokens < 1 || c->max_topk < 1) return false;
  if (static_cast<int64_t>(c->max_pages) * c->num_heads * kBlock >= (1ll << 31)) return false;
  if (c->lin_mode != HSA_LIN_NONE && c->lin_mode != HSA_LIN_STATE && c->lin_mode != HSA_LIN_LINFORMER)
    return false;
  if (c->lin_mode == HSA_LIN_LINFORMER) {
    if (c->head_dim != 128) return false;
    if (c->lin_rank < kBlock || c->lin_rank > 2048 || (c->lin_rank % kBlock) != 0) return false;  // whole compressed pages
    if (c->lin_seg_tokens < 1 || c->lin_seg_tokens > c->max_q_tokens) return false;
  }
  if (c->gate_act != 0 && c->gate_act != 1) return false;
  if (!(c->softmax_scale >= 0.f)) return false;
  if (c->split_blocks < 0) return false;
  if (c->feature_map != HSA_PHI_ELU1 && c->feature_map != HSA_PHI_RELU) return false;
  if ((c->flags & HSA_CFG_ADAPTIVE) && c->max_pages > 8192) return false;
  return true;
}

Layout make_layout(const hsa_config* c) {
  Layout L{};
  const size_t H = c->num_heads, D = c->head_dim, P = c->max_pages;
  size_t o = 0;
  L.slot_S = align_up(H * D * D * 4, 1024);
  L.slot_z = align_up(H * D * 4, 1024);
  L.S = o;      o += 2 * L.slot_S;
  L.z = o;      o += 2 * L.slot_z;
  L.hilo = o;   o = align_up(o + H * 4 * D * D * 2, 1024);
  L.zop = o;    o = align_up(o + H * 2 * kZopBytes, 1024);
  L.ksum_saved = o; o = align_up(o + H * D * 4, 1024);
  L.ksum = o;   o = align_up(o + H * P * D * 4, 1024);
  L.state_total = o;
  const size_t tiles = (static_cast<size_t>(c->max_q_tokens) + kTileM - 1) / kTileM;
  o = 0;
  L.status = o;     o = align_up(o + 16, 256);
  L.page_table = o; o = align_up(o + P * 4, 256);
  L.qpart = o;      o = align_up(o + tiles * H * D * 4, 256);
  L.keys = o;       o = align_up(o + H * tiles * P * 4, 256);
  L.spart = o;      o = align_up(o + H * kStateSplitMax * (D * D + D) * 4, 256);
  if (c->flags & HSA_CFG_CAUSAL) {
    L.lin_num = o;  o = align_up(o + static_cast<size_t>(c->max_q_tokens) * H * D * 4, 256);
    L.lin_den = o;  o = align_up(o + static_cast<size_t>(c->max_q_tokens) * H * 4, 256);
  }
  if (c->flags & HSA_CFG_ADAPTIVE) {
    L.ad_w = o;    o = align_up(o + H * tiles * P * 8, 256);
    L.ad_idx = o;  o = align_up(o + H * tiles * P * 4, 256);
    L.ad_gini = o; o = align_up(o + H * tiles * 8, 256);
    L.ad_wsum = o; o = align_up(o + H * tiles * 8, 256);
  }
  if (c->lin_mode == HSA_LIN_LINFORMER) {
    const size_t max_segs = (P * kBlock) / static_cast<size_t>(c->lin_seg_tokens);
    L.n_cpages = (max_segs > 0 ? max_segs : 1) * (static_cast<size_t>(c->lin_rank) / kBlock);
    L.cpool = L.n_cpages * H * kBlock * D * 2;
    L.ctable = o; o = align_up(o + L.n_cpages * 4, 256);
    L.csel = o;   o = align_up(o + H * L.n_cpages * 4, 256);
    L.ccnt = o;   o = align_up(o + H * 4, 256);
    L.olin = o;   o = align_up(o + static_cast<size_t>(c->max_q_tokens) * H * D * 2, 256);
  }
  // split tiles of the forward kernel
  L.split_blocks = c->split_blocks > 0 ? c->split_blocks : 256;
  L.split_blocks += L.split_blocks & 1;  // whole two-page steps
  L.fwd_splits = (c->max_topk + L.split_blocks - 1) / L.split_blocks;
  if (L.fwd_splits > kFwdSplitMax) L.fwd_splits = kFwdSplitMax;
  if (L.fwd_splits > 1) {
    const size_t slots = tiles * H * static_cast<size_t>(L.fwd_splits);
    L.part_o = o;      o = align_up(o + slots * kTileM * D * 4, 256);
    L.part_l = o;      o = align_up(o + slots * kTileM * 4, 256);
    L.part_ref = o;    o = align_up(o + slots * kTileM * 4, 256);
    L.part_ticket = o; o = align_up(o + tiles * H * 4, 256);
  }
  L.ws_total = o;
  return L;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

struct hsa_ctx {
  unsigned long long wait_ns;  // bound of the selection kernel's grid-barrier waits
  hsa_config cfg;
  hsa_buffers buf;
  Layout lay;
  float scale;
  int64_t n_tokens;
  int32_t last_append;  // tokens of the most recent append (0 after a rewind)
  int cur_slot;         // state slot that holds the running state of the current history
  int64_t tail_saved_for;  // history length whose tail-block key sum sits in the saved-tail buffer (-1: none)
  int nsm;
  CUtensorMap tm_k, tm_v, tm_state, tm_kc, tm_vc, tm_olin, tm_ek, tm_ev;
  int32_t n_segs;  // Linformer: complete segments compressed so far
  std::vector<int32_t> page_table_host;  // history block -> physical page
  std::vector<uint8_t> resident;         // per history block: tiles present in the pool (tier migration)
  int last_cuda_error;
};

namespace {

int cuda_fail(hsa_ctx* ctx, cudaError_t e) {
  if (ctx) ctx->last_cuda_error = static_cast<int>(e);
  return HSA_ERR_CUDA;
}

int encode_2d_rows(CUtensorMap* tm, void* base, uint64_t rows, int D) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return HSA_ERR_CUDA;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(D), rows};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(D) * 2};
  cuuint32_t box[2] = {64, 64};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? HSA_OK : HSA_ERR_CUDA;
}

int encode_q(CUtensorMap* tm, const void* q, int n_q, int H, int D, int64_t ts, int64_t hs,
             int box_rows = kTileM) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return HSA_ERR_CUDA;
  cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(H),
                        static_cast<cuuint64_t>(n_q)};
  cuuint64_t strides[2] = {static_cast<cuuint64_t>(hs) * 2, static_cast<cuuint64_t>(ts) * 2};
  cuuint32_t box[3] = {64, 1, static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides, box,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? HSA_OK : HSA_ERR_CUDA;
}

int encode_proj(CUtensorMap* tm, const void* e, int H, int seg_tokens, int rank) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return HSA_ERR_CUDA;
  cuuint64_t dims[3] = {static_cast<cuuint64_t>(rank), static_cast<cuuint64_t>(seg_tokens), static_cast<cuuint64_t>(H)};
  cuuint64_t strides[2] = {static_cast<cuuint64_t>(rank) * 2, static_cast<cuuint64_t>(seg_tokens) * rank * 2};
  cuuint32_t box[3] = {64, 64, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(e), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? HSA_OK : HSA_ERR_CUDA;
}

bool tensor_args_ok(const hsa_ctx* ctx, const void* p, int64_t ts, int64_t hs) {
  const int D = ctx->cfg.head_dim, H = ctx->cfg.num_heads;
  if (!p || !aligned(p, 16)) return false;
  if (ts <= 0 || hs <= 0 || (ts % 8) != 0 || (hs % 8) != 0) return false;
  if (hs < D || ts < D) return false;
  (void)H;
  return true;
}

}  // namespace

extern "C" {

int hsa_query_sizes(const hsa_config* cfg, hsa_sizes* out) {
  if (!config_ok(cfg) || !out) return HSA_ERR_INVALID_ARG;
  const Layout L = make_layout(cfg);
  const size_t pool = static_cast<size_t>(cfg->max_pages) * cfg->num_heads * kBlock * cfg->head_dim * 2;
  out->k_pool = pool;
  out->v_pool = pool;
  out->state = L.state_total;
  out->workspace = L.ws_total;
  out->kc_pool = L.cpool;
  out->vc_pool = L.cpool;
  return HSA_OK;
}

int hsa_create(hsa_ctx** out, const hsa_config* cfg, const hsa_buffers* bufs,
               const int32_t* page_alloc_order_host) {
  if (!out) return HSA_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config_ok(cfg) || !bufs) return HSA_ERR_INVALID_ARG;
  if (!bufs->k_pool || !bufs->v_pool || !bufs->state || !bufs->workspace) return HSA_ERR_INVALID_ARG;
  if (!aligned(bufs->k_pool, 256) || !aligned(bufs->v_pool, 256) || !aligned(bufs->state, 256) ||
      !aligned(bufs->workspace, 256))
    return HSA_ERR_INVALID_ARG;
  std::vector<int32_t> pt(cfg->max_pages);
  if (page_alloc_order_host) {
    std::vector<char> seen(cfg->max_pages, 0);
    for (int i = 0; i < cfg->max_pages; ++i) {
      const int32_t v = page_alloc_order_host[i];
      if (v < 0 || v >= cfg->max_pages || seen[v]) return HSA_ERR_INVALID_ARG;  // not a permutation
      seen[v] = 1;
      pt[i] = v;
    }
  } else {
    for (int i = 0; i < cfg->max_pages; ++i) pt[i] = i;
  }
  hsa_ctx* ctx = new (std::nothrow) hsa_ctx();
  if (!ctx) return HSA_ERR_INVALID_ARG;
  ctx->cfg = *cfg;
  ctx->buf = *bufs;
  ctx->lay = make_layout(cfg);
  ctx->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale
                                        : 1.0f / std::sqrt(static_cast<float>(cfg->head_dim));
  ctx->n_tokens = 0;
  ctx->last_append = 0;
  ctx->last_cuda_error = 0;
  ctx->n_segs = 0;
  ctx->cur_slot = 0;
  ctx->tail_saved_for = -1;
  ctx->wait_ns = 2000000000ull;
  ctx->page_table_host = pt;
  ctx->resident.assign(static_cast<size_t>(cfg->max_pages), 1);
  const bool linformer = cfg->lin_mode == HSA_LIN_LINFORMER;
  if (linformer) {
    if (!bufs->kc_pool || !bufs->vc_pool || !bufs->e_k || !bufs->e_v || !aligned(bufs->kc_pool, 256) ||
        !aligned(bufs->vc_pool, 256) || !aligned(bufs->e_k, 16) || !aligned(bufs->e_v, 16)) {
      delete ctx;
      return HSA_ERR_INVALID_ARG;
    }
  }

  cudaError_t e;
  int dev = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) { delete ctx; return HSA_ERR_CUDA; }
  int cc_major = 0;
  cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev);
  cudaDeviceGetAttribute(&ctx->nsm, cudaDevAttrMultiProcessorCount, dev);
  if (cc_major != 10) { delete ctx; return HSA_ERR_UNSUPPORTED; }  // sm_100a only, no fallback
  uint8_t* ws = static_cast<uint8_t*>(bufs->workspace);
  e = cudaMemcpy(ws + ctx->lay.page_table, pt.data(), pt.size() * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemset(ws + ctx->lay.status, 0, 16);
  if (e == cudaSuccess && ctx->lay.fwd_splits > 1)
    e = cudaMemset(ws + ctx->lay.part_ticket, 0,
                   static_cast<size_t>((cfg->max_q_tokens + kTileM - 1) / kTileM) * cfg->num_heads * 4);
  if (e == cudaSuccess) e = cudaMemset(bufs->state, 0, ctx->lay.state_total);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = forward_init();
  if (e == cudaSuccess) e = append_init();
  if (e == cudaSuccess) e = linear_only_init();
  if (e == cudaSuccess && linformer) {
    e = linformer_init();
    // identity page table and "every page" selection of the compressed pool
    std::vector<int32_t> iota(ctx->lay.n_cpages);
    for (size_t i = 0; i < iota.size(); ++i) iota[i] = static_cast<int32_t>(i);
    if (e == cudaSuccess)
      e = cudaMemcpy(ws + ctx->lay.ctable, iota.data(), iota.size() * 4, cudaMemcpyHostToDevice);
    for (int hh = 0; hh < cfg->num_heads && e == cudaSuccess; ++hh)
      e = cudaMemcpy(ws + ctx->lay.csel + static_cast<size_t>(hh) * iota.size() * 4, iota.data(),
                     iota.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(ws + ctx->lay.ccnt, 0, static_cast<size_t>(cfg->num_heads) * 4);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
  }
  if (e != cudaSuccess) { delete ctx; return HSA_ERR_CUDA; }
  const int D = cfg->head_dim;
  const uint64_t pool_rows = static_cast<uint64_t>(cfg->max_pages) * cfg->num_heads * kBlock;
  int r = encode_2d_rows(&ctx->tm_k, bufs->k_pool, pool_rows, D);
  if (r == HSA_OK) r = encode_2d_rows(&ctx->tm_v, bufs->v_pool, pool_rows, D);
  if (r == HSA_OK)
    r = encode_2d_rows(&ctx->tm_state, static_cast<uint8_t*>(bufs->state) + ctx->lay.hilo,
                       static_cast<uint64_t>(cfg->num_heads) * 4 * D, D);
  if (r == HSA_OK && linformer) {
    const uint64_t crows = static_cast<uint64_t>(ctx->lay.n_cpages) * cfg->num_heads * kBlock;
    r = encode_2d_rows(&ctx->tm_kc, bufs->kc_pool, crows, D);
    if (r == HSA_OK) r = encode_2d_rows(&ctx->tm_vc, bufs->vc_pool, crows, D);
    // projection weights [H][seg_tokens][rank]: boxes of 64 r x 64 tokens of one head
    if (r == HSA_OK) r = encode_proj(&ctx->tm_ek, bufs->e_k, cfg->num_heads, cfg->lin_seg_tokens, cfg->lin_rank);
    if (r == HSA_OK) r = encode_proj(&ctx->tm_ev, bufs->e_v, cfg->num_heads, cfg->lin_seg_tokens, cfg->lin_rank);
  }
  if (r != HSA_OK) { delete ctx; return r; }
  *out = ctx;
  return HSA_OK;
}

int hsa_append_kv(hsa_ctx* ctx, const void* k, const void* v, int32_t n_tokens, int64_t tok_stride,
                  int64_t head_stride, void* stream) {
  if (!ctx) return HSA_ERR_INVALID_ARG;
  if (n_tokens < 1 || n_tokens > ctx->cfg.max_q_tokens) return HSA_ERR_INVALID_ARG;
  if (!tensor_args_ok(ctx, k, tok_stride, head_stride) || !tensor_args_ok(ctx, v, tok_stride, head_stride))
    return HSA_ERR_INVALID_ARG;
  const int64_t n1 = ctx->n_tokens + n_tokens;
  if ((n1 + kBlock - 1) / kBlock > ctx->cfg.max_pages) return HSA_ERR_OUT_OF_PAGES;
  uint8_t* stt = static_cast<uint8_t*>(ctx->buf.state);
  uint8_t* ws = static_cast<uint8_t*>(ctx->buf.workspace);
  AppendArgs a{};
  a.k = static_cast<const __nv_bfloat16*>(k);
  a.v = static_cast<const __nv_bfloat16*>(v);
  a.n_new = n_tokens;
  a.tok_stride = tok_stride;
  a.head_stride = head_stride;
  a.n0 = ctx->n_tokens;
  a.H = ctx->cfg.num_heads;
  a.D = ctx->cfg.head_dim;
  a.max_pages = ctx->cfg.max_pages;
  a.page_table = reinterpret_cast<const int32_t*>(ws + ctx->lay.page_table);
  a.k_pool = static_cast<__nv_bfloat16*>(ctx->buf.k_pool);
  a.v_pool = static_cast<__nv_bfloat16*>(ctx->buf.v_pool);
  a.ksum = reinterpret_cast<float*>(stt + ctx->lay.ksum);
  for (int sl = 0; sl < 2; ++sl) {
    a.S[sl] = reinterpret_cast<float*>(stt + ctx->lay.S + sl * ctx->lay.slot_S);
    a.z[sl] = reinterpret_cast<float*>(stt + ctx->lay.z + sl * ctx->lay.slot_z);
  }
  a.src_slot = ctx->cur_slot;
  a.ksum_saved = reinterpret_cast<float*>(stt + ctx->lay.ksum_saved);
  a.tail_from_saved = (ctx->n_tokens % kBlock) != 0 && ctx->tail_saved_for == ctx->n_tokens;
  a.hilo = reinterpret_cast<__nv_bfloat16*>(stt + ctx->lay.hilo);
  a.zop = stt + ctx->lay.zop;
  a.spart = reinterpret_cast<float*>(ws + ctx->lay.spart);
  int nsplit = ctx->nsm / a.H;
  if (nsplit < 1) nsplit = 1;
  if (nsplit > kStateSplitMax) nsplit = kStateSplitMax;
  const int by_tokens = (n_tokens + 31) / 32;
  if (nsplit > by_tokens) nsplit = by_tokens;
  a.nsplit = nsplit;
  a.lin_state = ctx->cfg.lin_mode == HSA_LIN_STATE;
  a.relu = ctx->cfg.feature_map == HSA_PHI_RELU;
  a.status = reinterpret_cast<int32_t*>(ws + ctx->lay.status);
  const bool linformer = ctx->cfg.lin_mode == HSA_LIN_LINFORMER;
  if (linformer && (n_tokens != ctx->cfg.lin_seg_tokens || ctx->n_tokens != static_cast<int64_t>(ctx->n_segs) * n_tokens))
    return HSA_ERR_UNSUPPORTED;  // this mode appends whole segments only
  AppendMaps maps;
  const bool fused = a.D == 128 && a.lin_state;
  if (fused || linformer) {
    if (encode_q(&maps.kin, k, n_tokens, a.H, a.D, tok_stride, head_stride, kBlock) != HSA_OK ||
        encode_q(&maps.vin, v, n_tokens, a.H, a.D, tok_stride, head_stride, kBlock) != HSA_OK)
      return HSA_ERR_CUDA;
    maps.kpool = ctx->tm_k;
    maps.vpool = ctx->tm_v;
  }
  cudaError_t e = cudaSuccess;
  if (!linformer) {
    e = launch_append(a, fused ? &maps : nullptr, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
  }
  if (linformer) {
    LinformerArgs la{};
    la.k = a.k;
    la.v = a.v;
    la.tok_stride = tok_stride;
    la.head_stride = head_stride;
    la.e_k = static_cast<const __nv_bfloat16*>(ctx->buf.e_k);
    la.e_v = static_cast<const __nv_bfloat16*>(ctx->buf.e_v);
    la.kc_pool = static_cast<__nv_bfloat16*>(ctx->buf.kc_pool);
    la.vc_pool = static_cast<__nv_bfloat16*>(ctx->buf.vc_pool);
    la.ccnt = reinterpret_cast<int32_t*>(ws + ctx->lay.ccnt);
    la.H = a.H;
    la.rank = ctx->cfg.lin_rank;
    la.seg_tokens = ctx->cfg.lin_seg_tokens;
    la.seg_index = ctx->n_segs;
    la.status = a.status;
    e = launch_linformer_compress(la, ctx->tm_ek, ctx->tm_ev, maps.kin, maps.vin, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    // pages and key sums of the chunk: launched behind the compression kernel, runs beside it (the
    // two write nothing in common) and ends after it
    a.beside_prior = 1;
    e = launch_append(a, nullptr, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->n_segs += 1;
  }
  for (int64_t b = ctx->n_tokens / kBlock; b <= (n1 - 1) / kBlock; ++b) ctx->resident[static_cast<size_t>(b)] = 1;
  if (ctx->n_tokens % kBlock) ctx->tail_saved_for = ctx->n_tokens;
  if (a.lin_state) ctx->cur_slot ^= 1;  // the append wrote the other slot
  ctx->n_tokens = n1;
  ctx->last_append = n_tokens;
  return HSA_OK;
}

int hsa_select_blocks(hsa_ctx* ctx, const void* q, int32_t n_q, int64_t tok_stride, int64_t head_stride,
                      int64_t q_pos0, int32_t causal, const int32_t* budgets_dev,
                      int32_t q_group_tokens, int32_t* sel_idx_dev, int32_t* sel_cnt_dev,
                      void* stream) {
  return hsa_select_blocks_ex(ctx, q, n_q, tok_stride, head_stride, q_pos0, causal, budgets_dev, q_group_tokens,
                              nullptr, sel_idx_dev, sel_cnt_dev, stream);
}

int hsa_select_blocks_ex(hsa_ctx* ctx, const void* q, int32_t n_q, int64_t tok_stride, int64_t head_stride,
                         int64_t q_pos0, int32_t causal, const int32_t* budgets_dev,
                         int32_t q_group_tokens, const hsa_select_opts* opts, int32_t* sel_idx_dev,
                         int32_t* sel_cnt_dev, void* stream) {
  if (!ctx) return HSA_ERR_INVALID_ARG;
  if (opts && (opts->inter_block_pages < 0 || opts->inter_block_pages > 2)) return HSA_ERR_INVALID_ARG;
  if (n_q < 1 || n_q > ctx->cfg.max_q_tokens) return HSA_ERR_INVALID_ARG;
  if (!tensor_args_ok(ctx, q, tok_stride, head_stride)) return HSA_ERR_INVALID_ARG;
  if (!budgets_dev || !sel_idx_dev || !sel_cnt_dev) return HSA_ERR_INVALID_ARG;
  if (q_group_tokens < 0 || (q_group_tokens % kTileM) != 0) return HSA_ERR_INVALID_ARG;
  const int64_t nblk = (ctx->n_tokens + kBlock - 1) / kBlock;
  if (nblk * 4 > 200 * 1024) return HSA_ERR_UNSUPPORTED;  // keys of one head must fit shared memory
  uint8_t* stt = static_cast<uint8_t*>(ctx->buf.state);
  uint8_t* ws = static_cast<uint8_t*>(ctx->buf.workspace);
  SelectArgs a{};
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.n_q = n_q;
  a.tok_stride = tok_stride;
  a.head_stride = head_stride;
  a.q_pos0 = q_pos0;
  a.causal = causal != 0;
  a.n_tokens = ctx->n_tokens;
  a.H = ctx->cfg.num_heads;
  a.D = ctx->cfg.head_dim;
  a.max_pages = ctx->cfg.max_pages;
  a.ksum = reinterpret_cast<const float*>(stt + ctx->lay.ksum);
  a.budgets = budgets_dev;
  a.group_tokens = q_group_tokens;
  a.n_groups = q_group_tokens > 0 ? (n_q + q_group_tokens - 1) / q_group_tokens : 1;
  a.scale = ctx->scale;
  a.qpart = reinterpret_cast<float*>(ws + ctx->lay.qpart);
  a.keys = reinterpret_cast<uint32_t*>(ws + ctx->lay.keys);
  a.sel_idx = sel_idx_dev;
  a.sel_cnt = sel_cnt_dev;
  a.kcap = ctx->cfg.max_topk;
  a.status = reinterpret_cast<int32_t*>(ws + ctx->lay.status);
  a.barrier = reinterpret_cast<unsigned*>(ws + ctx->lay.status + 8);
  a.wait_ns = ctx->wait_ns;
  a.use_clusters = (ctx->cfg.flags & HSA_CFG_GRID_BARRIER_SELECT) ? 0 : 1;
  if (opts) {
    a.inter_pages = opts->inter_block_pages;
    a.intra_first_page1 = opts->intra_first_page >= 0 ? static_cast<int64_t>(opts->intra_first_page) + 1 : 0;
    a.intra_budgets = opts->intra_budgets_dev;
    if (opts->kv_pages_dev) {
      if (opts->n_kv_pages < 0 || opts->n_kv_pages > 64 || opts->kv_page_blocks < 1) return HSA_ERR_INVALID_ARG;
      a.kv_pages = opts->kv_pages_dev;
      a.n_kv_pages = opts->n_kv_pages;
      a.kv_page_blocks = opts->kv_page_blocks;
    }
  }
  cudaError_t e = launch_select(a, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  return HSA_OK;
}

int hsa_select_blocks_adaptive(hsa_ctx* ctx, const void* q, int32_t n_q, int64_t tok_stride,
                               int64_t head_stride, int64_t q_pos0, int32_t causal, float tau_min,
                               float tau_max, int32_t q_group_tokens, int32_t* sel_idx_dev,
                               int32_t* sel_cnt_dev, float* gini_tau_out_dev, void* stream) {
  if (!ctx) return HSA_ERR_INVALID_ARG;
  if (!(ctx->cfg.flags & HSA_CFG_ADAPTIVE)) return HSA_ERR_UNSUPPORTED;
  if (n_q < 1 || n_q > ctx->cfg.max_q_tokens) return HSA_ERR_INVALID_ARG;
  if (!tensor_args_ok(ctx, q, tok_stride, head_stride)) return HSA_ERR_INVALID_ARG;
  if (!sel_idx_dev || !sel_cnt_dev) return HSA_ERR_INVALID_ARG;
  if (q_group_tokens < 0 || (q_group_tokens % kTileM) != 0) return HSA_ERR_INVALID_ARG;
  if (!(tau_min >= 0.f) || !(tau_max <= 1.f) || !(tau_min <= tau_max)) return HSA_ERR_INVALID_ARG;
  const int64_t nblk = (ctx->n_tokens + kBlock - 1) / kBlock;
  if (nblk > 8192) return HSA_ERR_UNSUPPORTED;
  uint8_t* stt = static_cast<uint8_t*>(ctx->buf.state);
  uint8_t* ws = static_cast<uint8_t*>(ctx->buf.workspace);
  SelectArgs a{};
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.n_q = n_q;
  a.tok_stride = tok_stride;
  a.head_stride = head_stride;
  a.q_pos0 = q_pos0;
  a.causal = causal != 0;
  a.n_tokens = ctx->n_tokens;
  a.H = ctx->cfg.num_heads;
  a.D = ctx->cfg.head_dim;
  a.max_pages = ctx->cfg.max_pages;
  a.ksum = reinterpret_cast<const float*>(stt + ctx->lay.ksum);
  a.budgets = nullptr;
  a.group_tokens = q_group_tokens;
  a.n_groups = q_group_tokens > 0 ? (n_q + q_group_tokens - 1) / q_group_tokens : 1;
  a.scale = ctx->scale;
  a.qpart = reinterpret_cast<float*>(ws + ctx->lay.qpart);
  a.keys = reinterpret_cast<uint32_t*>(ws + ctx->lay.keys);
  a.sel_idx = sel_idx_dev;
  a.sel_cnt = sel_cnt_dev;
  a.kcap = ctx->cfg.max_topk;
  a.status = reinterpret_cast<int32_t*>(ws + ctx->lay.status);
  AdaptiveArgs ad{};
  ad.sorted_w = reinterpret_cast<double*>(ws + ctx->lay.ad_w);
  ad.sorted_idx = reinterpret_cast<int32_t*>(ws + ctx->lay.ad_idx);
  ad.gini_part = reinterpret_cast<double*>(ws + ctx->lay.ad_gini);
  ad.wsum = reinterpret_cast<double*>(ws + ctx->lay.ad_wsum);
  ad.tau_min = tau_min;
  ad.tau_max = tau_max;
  ad.gini_out = gini_tau_out_dev;
  cudaError_t e = launch_select_adaptive(a, ad, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  return HSA_OK;
}

int hsa_forward(hsa_ctx* ctx, const void* q, int32_t n_q, int64_t tok_stride, int64_t head_stride,
                int64_t q_pos0, int32_t causal, const int32_t* sel_idx_dev, const int32_t* sel_cnt_dev,
                int32_t q_group_tokens, const void* g_lin, const void* g_sp, int64_t gate_tok_stride,
                int64_t gate_head_stride, int64_t gate_dim_stride, void* out, int64_t out_tok_stride,
                int64_t out_head_stride, uint32_t flags, void* stream) {
  if (!ctx) return HSA_ERR_INVALID_ARG;
  if (n_q < 1 || n_q > ctx->cfg.max_q_tokens) return HSA_ERR_INVALID_ARG;
  if (!tensor_args_ok(ctx, q, tok_stride, head_stride)) return HSA_ERR_INVALID_ARG;
  if (!tensor_args_ok(ctx, out, out_tok_stride, out_head_stride)) return HSA_ERR_INVALID_ARG;
  if (q_group_tokens < 0 || (q_group_tokens % kTileM) != 0) return HSA_ERR_INVALID_ARG;
  if (flags & ~(HSA_FWD_NO_LINEAR | HSA_FWD_NO_SPARSE)) return HSA_ERR_INVALID_ARG;
  const bool do_sparse = !(flags & HSA_FWD_NO_SPARSE);
  const bool do_linear = !(flags & HSA_FWD_NO_LINEAR) && ctx->cfg.lin_mode == HSA_LIN_STATE;
  const bool do_linformer = !(flags & HSA_FWD_NO_LINEAR) && ctx->cfg.lin_mode == HSA_LIN_LINFORMER &&
                            ctx->n_segs > 0;
  if (do_linformer && causal) return HSA_ERR_UNSUPPORTED;
  if (do_sparse && (!sel_idx_dev || !sel_cnt_dev)) return HSA_ERR_INVALID_ARG;
  if ((g_lin || g_sp) && (gate_tok_stride < 0 || gate_head_stride < 0 || gate_dim_stride < 0))
    return HSA_ERR_INVALID_ARG;
  const bool causal_lin = causal && do_linear;
  if (causal_lin) {
    if (!(ctx->cfg.flags & HSA_CFG_CAUSAL)) return HSA_ERR_UNSUPPORTED;
    if (q_pos0 + n_q != ctx->n_tokens || n_q != ctx->last_append) return HSA_ERR_UNSUPPORTED;
  }
  const int D = ctx->cfg.head_dim, H = ctx->cfg.num_heads;
  uint8_t* stt = static_cast<uint8_t*>(ctx->buf.state);
  uint8_t* ws = static_cast<uint8_t*>(ctx->buf.workspace);
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  CUtensorMap tm_q;
  int r = encode_q(&tm_q, q, n_q, H, D, tok_stride, head_stride);
  if (r != HSA_OK) return r;

  CUtensorMap tm_out;  // same geometry as q: the kernel stores whole [128 rows x 64 dims] tiles
  r = encode_q(&tm_out, out, n_q, H, D, out_tok_stride, out_head_stride);
  if (r != HSA_OK) return r;

  FwdParams p{};
  p.n_q = n_q;
  p.H = H;
  p.n_tokens = ctx->n_tokens;
  p.q_pos0 = q_pos0;
  p.causal = causal != 0;
  p.sel_idx = sel_idx_dev;
  p.sel_cnt = sel_cnt_dev;
  p.kcap = ctx->cfg.max_topk;
  p.group_tokens = q_group_tokens;
  p.n_groups = q_group_tokens > 0 ? (n_q + q_group_tokens - 1) / q_group_tokens : 1;
  p.page_table = reinterpret_cast<const int32_t*>(ws + ctx->lay.page_table);
  p.n_blocks = static_cast<int>((ctx->n_tokens + kBlock - 1) / kBlock);
  p.state_slot = ctx->cur_slot ^ (causal_lin ? 1 : 0);  // causal: the state before the chunk's own append
  p.z = reinterpret_cast<const float*>(stt + ctx->lay.z + p.state_slot * ctx->lay.slot_z);
  p.zop = stt + ctx->lay.zop;
  p.g_lin = static_cast<const __nv_bfloat16*>(g_lin);
  p.g_sp = static_cast<const __nv_bfloat16*>(g_sp);
  p.g_ts = gate_tok_stride;
  p.g_hs = gate_head_stride;
  p.g_ds = gate_dim_stride;
  p.gate_act = ctx->cfg.gate_act;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.o_ts = out_tok_stride;
  p.o_hs = out_head_stride;
  p.scale_log2 = ctx->scale * 1.4426950408889634f;
  p.flags = flags;
  p.do_linear = do_linear;
  p.relu = ctx->cfg.feature_map == HSA_PHI_RELU;
  p.do_sparse = do_sparse;
  p.status = reinterpret_cast<int32_t*>(ws + ctx->lay.status);
  p.max_splits = 1;
  p.nsm = ctx->nsm;
  p.k_pool = static_cast<const uint8_t*>(ctx->buf.k_pool);
  p.v_pool = static_cast<const uint8_t*>(ctx->buf.v_pool);
  if (do_sparse && ctx->lay.fwd_splits > 1) {
    p.max_splits = ctx->lay.fwd_splits;
    p.split_blocks = ctx->lay.split_blocks;
    p.part_o = reinterpret_cast<float*>(ws + ctx->lay.part_o);
    p.part_l = reinterpret_cast<float*>(ws + ctx->lay.part_l);
    p.part_ref = reinterpret_cast<float*>(ws + ctx->lay.part_ref);
    p.part_ticket = reinterpret_cast<int32_t*>(ws + ctx->lay.part_ticket);
  }
  if (causal_lin) {
    CausalLinArgs c{};
    c.q = static_cast<const __nv_bfloat16*>(q);
    c.n_q = n_q;
    c.q_ts = tok_stride;
    c.q_hs = head_stride;
    c.k_pool = static_cast<const __nv_bfloat16*>(ctx->buf.k_pool);
    c.v_pool = static_cast<const __nv_bfloat16*>(ctx->buf.v_pool);
    c.page_table = p.page_table;
    c.q_pos0 = q_pos0;
    c.n_tokens = ctx->n_tokens;
    c.H = H;
    c.D = D;
    c.relu = p.relu;
    c.lin_num = reinterpret_cast<float*>(ws + ctx->lay.lin_num);
    c.lin_den = reinterpret_cast<float*>(ws + ctx->lay.lin_den);
    cudaError_t e = launch_causal_linear(c, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    p.lin_num = c.lin_num;
    p.lin_den = c.lin_den;
  }
  if (do_linformer && p.max_splits == 1 && D == 128) {
    // one launch: the kernel's loop runs over the compressed pool first (its own accumulator,
    // exponent reference and row sums), then over the selected pages, and merges in its epilogue
    p.lf_table = reinterpret_cast<const int32_t*>(ws + ctx->lay.ctable);
    p.lf_pages = static_cast<int>(static_cast<int64_t>(ctx->n_segs) * ctx->cfg.lin_rank / kBlock);
    p.do_linear = 1;  // the compressed segment is this launch's linear branch
    cudaError_t ef = launch_forward(p, D, tm_q, ctx->tm_k, ctx->tm_v, ctx->tm_state, tm_out, st, &ctx->tm_kc, &ctx->tm_vc);
    if (ef != cudaSuccess) return cuda_fail(ctx, ef);
    return HSA_OK;
  }
  if (do_linformer) {
    // long lists split over CTAs: two launches.  Pass 1: plain softmax attention of the chunk over
    // every compressed row -> O_lin (bf16) in the workspace; pass 2 below picks it up in its epilogue
    uint8_t* olin = ws + ctx->lay.olin;
    CUtensorMap tm_olin;
    r = encode_q(&tm_olin, olin, n_q, H, D, static_cast<int64_t>(H) * D, D);
    if (r != HSA_OK) return r;
    FwdParams p1{};
    p1.n_q = n_q;
    p1.H = H;
    p1.n_tokens = static_cast<int64_t>(ctx->n_segs) * ctx->cfg.lin_rank;
    p1.q_pos0 = p1.n_tokens;
    p1.causal = 0;
    p1.sel_idx = reinterpret_cast<const int32_t*>(ws + ctx->lay.csel);
    p1.sel_cnt = reinterpret_cast<const int32_t*>(ws + ctx->lay.ccnt);
    p1.kcap = static_cast<int>(ctx->lay.n_cpages);
    p1.group_tokens = 0;
    p1.n_groups = 1;
    p1.page_table = reinterpret_cast<const int32_t*>(ws + ctx->lay.ctable);
    p1.n_blocks = static_cast<int>(p1.n_tokens / kBlock);
    p1.z = p.z;
    p1.out = reinterpret_cast<__nv_bfloat16*>(olin);
    p1.o_ts = static_cast<int64_t>(H) * D;
    p1.o_hs = D;
    p1.scale_log2 = p.scale_log2;
    p1.do_linear = 0;
    p1.do_sparse = 1;
    p1.max_splits = 1;
    p1.status = p.status;
    cudaError_t e1 = launch_forward(p1, D, tm_q, ctx->tm_kc, ctx->tm_vc, ctx->tm_state, tm_olin, st);
    if (e1 != cudaSuccess) return cuda_fail(ctx, e1);
    p.ext_lin = reinterpret_cast<const __nv_bfloat16*>(olin);
  }
  cudaError_t e;
  if (D == 128 && do_linear && !do_sparse && !p.ext_lin)
    e = launch_linear_only(p, ctx->nsm, tm_q, ctx->tm_state, tm_out, st);  // nothing but Q in, out out
  else
    e = launch_forward(p, D, tm_q, ctx->tm_k, ctx->tm_v, ctx->tm_state, tm_out, st);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  return HSA_OK;
}

int hsa_retrieve_kv_pages(hsa_ctx* ctx, const void* q, int32_t n_q, int64_t tok_stride, int64_t head_stride,
                          int32_t kv_page_blocks, int32_t top_kp, int32_t* page_ids_dev, float* scores_dev,
                          int32_t* n_out_host, void* stream) {
  if (!ctx) return HSA_ERR_INVALID_ARG;
  if (n_q < 1 || n_q > ctx->cfg.max_q_tokens) return HSA_ERR_INVALID_ARG;
  if (!tensor_args_ok(ctx, q, tok_stride, head_stride)) return HSA_ERR_INVALID_ARG;
  if (kv_page_blocks < 1 || top_kp < 0 || top_kp > 64 || !page_ids_dev) return HSA_ERR_INVALID_ARG;
  const int64_t nblk = (ctx->n_tokens + kBlock - 1) / kBlock;
  const int64_t n_pages = (nblk + kv_page_blocks - 1) / kv_page_blocks;
  if (n_pages > 2048) return HSA_ERR_UNSUPPORTED;
  if (n_out_host) *n_out_host = static_cast<int32_t>(n_pages < top_kp ? n_pages : top_kp);
  if (n_pages == 0 || top_kp == 0) return HSA_OK;
  uint8_t* stt = static_cast<uint8_t*>(ctx->buf.state);
  uint8_t* ws = static_cast<uint8_t*>(ctx->buf.workspace);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  SelectArgs sa{};
  sa.q = static_cast<const __nv_bfloat16*>(q);
  sa.n_q = n_q;
  sa.tok_stride = tok_stride;
  sa.head_stride = head_stride;
  sa.H = ctx->cfg.num_heads;
  sa.D = ctx->cfg.head_dim;
  sa.qpart = reinterpret_cast<float*>(ws + ctx->lay.qpart);
  cudaError_t e = launch_qsum(sa, st);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  RetrieveArgs ra{};
  ra.n_q = n_q;
  ra.H = sa.H;
  ra.D = sa.D;
  ra.max_pages = ctx->cfg.max_pages;
  ra.n_tokens = ctx->n_tokens;
  ra.qpart = sa.qpart;
  ra.ksum = reinterpret_cast<const float*>(stt + ctx->lay.ksum);
  ra.kv_page_blocks = kv_page_blocks;
  ra.top_kp = top_kp;
  ra.scale = ctx->scale;
  ra.keys = reinterpret_cast<uint32_t*>(ws + ctx->lay.keys);
  ra.scores_out = scores_dev;
  ra.page_ids = page_ids_dev;
  e = launch_retrieve(ra, static_cast<int>(n_pages), st);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  return HSA_OK;
}

namespace {
// Copies the tiles of blocks [b0, b0 + n) between the pools and host buffers, one cudaMemcpyAsync
// per pool and run of physically adjacent pages.
int migrate_blocks(hsa_ctx* ctx, int32_t b0, int32_t n, void* host_k, void* host_v, bool to_host, void* stream) {
  if (!ctx || !host_k || !host_v || b0 < 0 || n < 0) return HSA_ERR_INVALID_ARG;
  const int64_t nblk = (ctx->n_tokens + kBlock - 1) / kBlock;
  if (static_cast<int64_t>(b0) + n > nblk) return HSA_ERR_INVALID_ARG;
  const size_t tile = static_cast<size_t>(ctx->cfg.num_heads) * kBlock * ctx->cfg.head_dim * 2;  // one page, one pool
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* pools[2] = {static_cast<uint8_t*>(ctx->buf.k_pool), static_cast<uint8_t*>(ctx->buf.v_pool)};
  uint8_t* hosts[2] = {static_cast<uint8_t*>(host_k), static_cast<uint8_t*>(host_v)};
  int32_t i = 0;
  while (i < n) {
    int32_t run = 1;
    const int32_t p_first = ctx->page_table_host[static_cast<size_t>(b0 + i)];
    while (i + run < n && ctx->page_table_host[static_cast<size_t>(b0 + i + run)] == p_first + run) ++run;
    for (int w = 0; w < 2; ++w) {
      uint8_t* dev = pools[w] + static_cast<size_t>(p_first) * tile;
      uint8_t* host = hosts[w] + static_cast<size_t>(i) * tile;
      cudaError_t e = to_host ? cudaMemcpyAsync(host, dev, run * tile, cudaMemcpyDeviceToHost, st)
                              : cudaMemcpyAsync(dev, host, run * tile, cudaMemcpyHostToDevice, st);
      if (e != cudaSuccess) return cuda_fail(ctx, e);
    }
    i += run;
  }
  for (int32_t b = b0; b < b0 + n; ++b) ctx->resident[static_cast<size_t>(b)] = to_host ? 0 : 1;
  return HSA_OK;
}
}  // namespace

int hsa_evict_blocks(hsa_ctx* ctx, int32_t first_block, int32_t n_blocks, void* host_k, void* host_v,
                     void* stream) {
  return migrate_blocks(ctx, first_block, n_blocks, host_k, host_v, true, stream);
}

int hsa_restore_blocks(hsa_ctx* ctx, int32_t first_block, int32_t n_blocks, const void* host_k,
                       const void* host_v, void* stream) {
  return migrate_blocks(ctx, first_block, n_blocks, const_cast<void*>(host_k), const_cast<void*>(host_v), false,
                        stream);
}

int hsa_block_resident(hsa_ctx* ctx, int32_t block, int32_t* resident_out) {
  if (!ctx || !resident_out || block < 0 || block >= ctx->cfg.max_pages) return HSA_ERR_INVALID_ARG;
  *resident_out = ctx->resident[static_cast<size_t>(block)];
  return HSA_OK;
}

int hsa_get_info(hsa_ctx* ctx, int64_t* n_tokens, int32_t* n_blocks) {
  if (!ctx) return HSA_ERR_INVALID_ARG;
  if (n_tokens) *n_tokens = ctx->n_tokens;
  if (n_blocks) *n_blocks = static_cast<int32_t>((ctx->n_tokens + kBlock - 1) / kBlock);
  return HSA_OK;
}

int hsa_rewind(hsa_ctx* ctx, int64_t n_tokens) {
  if (!ctx || n_tokens < 0 || n_tokens > ctx->n_tokens) return HSA_ERR_INVALID_ARG;
  if (ctx->cfg.lin_mode == HSA_LIN_LINFORMER) {
    if (n_tokens % ctx->cfg.lin_seg_tokens) return HSA_ERR_UNSUPPORTED;
    ctx->n_segs = static_cast<int32_t>(n_tokens / ctx->cfg.lin_seg_tokens);
  }
  // Undoing exactly the last append: the state before it is still in the other slot, and the key
  // sum its first block had before it is in the saved-tail buffer (the next append from this length
  // takes it from there), so nothing has to be restored.
  const bool undo = ctx->last_append > 0 && n_tokens == ctx->n_tokens - ctx->last_append;
  if (undo && ctx->cfg.lin_mode == HSA_LIN_STATE) ctx->cur_slot ^= 1;
  if (n_tokens < ctx->tail_saved_for) ctx->tail_saved_for = -1;
  ctx->n_tokens = n_tokens;
  ctx->last_append = 0;
  return HSA_OK;
}

int hsa_state_layout(hsa_ctx* ctx, size_t* off_S, size_t* off_z, size_t* off_ksum) {
  if (!ctx) return HSA_ERR_INVALID_ARG;
  if (off_S) *off_S = ctx->lay.S + ctx->cur_slot * ctx->lay.slot_S;
  if (off_z) *off_z = ctx->lay.z + ctx->cur_slot * ctx->lay.slot_z;
  if (off_ksum) *off_ksum = ctx->lay.ksum;
  return HSA_OK;
}

int hsa_workspace_layout(hsa_ctx* ctx, size_t* off_status, size_t* off_barrier) {
  if (!ctx) return HSA_ERR_INVALID_ARG;
  if (off_status) *off_status = ctx->lay.status;
  if (off_barrier) *off_barrier = ctx->lay.status + 8;
  return HSA_OK;
}

int hsa_set_wait_limit_ns(hsa_ctx* ctx, uint64_t wait_ns) {
  if (!ctx || wait_ns == 0) return HSA_ERR_INVALID_ARG;
  ctx->wait_ns = wait_ns;
  return HSA_OK;
}

int hsa_device_status(hsa_ctx* ctx, int32_t* status_out) {
  if (!ctx || !status_out) return HSA_ERR_INVALID_ARG;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  uint8_t* ws = static_cast<uint8_t*>(ctx->buf.workspace);
  int32_t v = 0;
  e = cudaMemcpy(&v, ws + ctx->lay.status, 4, cudaMemcpyDeviceToHost);
  if (e == cudaSuccess && v != 0) e = cudaMemset(ws + ctx->lay.status, 0, 4);
  // a grid barrier that ran out leaves its arrive count behind: both of its words start over
  if (e == cudaSuccess && v == HSA_ERR_DEVICE_TIMEOUT) e = cudaMemset(ws + ctx->lay.status + 8, 0, 8);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  *status_out = v;
  return HSA_OK;
}

int hsa_safe_pass_tiles(hsa_ctx* ctx, int64_t* count_out) {
  if (!ctx || !count_out) return HSA_ERR_INVALID_ARG;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  uint8_t* ws = static_cast<uint8_t*>(ctx->buf.workspace);
  int32_t v = 0;
  e = cudaMemcpy(&v, ws + ctx->lay.status + 4, 4, cudaMemcpyDeviceToHost);
  if (e == cudaSuccess && v != 0) e = cudaMemset(ws + ctx->lay.status + 4, 0, 4);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  *count_out = v;
  return HSA_OK;
}

int hsa_last_cuda_error(hsa_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

int hsa_destroy(hsa_ctx* ctx) {
  if (!ctx) return HSA_ERR_INVALID_ARG;
  delete ctx;
  return HSA_OK;
}

const char* hsa_status_string(int s) {
  switch (s) {
    case HSA_OK: return "ok";
    case HSA_ERR_INVALID_ARG: return "invalid argument";
    case HSA_ERR_OUT_OF_PAGES: return "out of pages";
    case HSA_ERR_UNSUPPORTED: return "unsupported";
    case HSA_ERR_CUDA: return "CUDA error";
    case HSA_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case HSA_ERR_DEVICE_BOUNDS: return "device-side index out of range";
    default: return "unknown status";
  }
}

}  // extern "C"
