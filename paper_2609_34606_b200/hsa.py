"""Thin Python binding over the HSA C-ABI library (libhsa.so).

Argument marshalling only: every step of the path (pool write, key sums, state
update, block scoring, top-k, both attention branches, the merge) runs in the
library's CUDA kernels.  torch is used for device memory and streams.  There is
no fallback: if libhsa.so is missing or fails to load, importing this module
raises.

The module-level functions carry the C names (hsa_create, hsa_append_kv,
hsa_select_blocks, hsa_forward, ...) and take torch tensors where the C ABI
takes device pointers; `HSAContext` bundles buffer allocation with them.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libhsa.so")

HSA_OK = 0
HSA_ERR_INVALID_ARG = -1
HSA_ERR_OUT_OF_PAGES = -2
HSA_ERR_UNSUPPORTED = -3
HSA_ERR_CUDA = -4
HSA_ERR_DEVICE_TIMEOUT = -5
HSA_ERR_DEVICE_BOUNDS = -6
HSA_LIN_NONE, HSA_LIN_STATE, HSA_LIN_LINFORMER = 0, 1, 2
HSA_PHI_ELU1, HSA_PHI_RELU = 0, 1
HSA_CFG_CAUSAL = 1
HSA_CFG_ADAPTIVE = 2
HSA_CFG_GRID_BARRIER_SELECT = 4
HSA_FWD_NO_LINEAR, HSA_FWD_NO_SPARSE = 1, 2
PAGE_TOKENS = 64
TILE_M = 128

EXPORTS = [
    "hsa_query_sizes", "hsa_create", "hsa_append_kv", "hsa_select_blocks", "hsa_select_blocks_ex",
    "hsa_select_blocks_adaptive", "hsa_retrieve_kv_pages", "hsa_evict_blocks", "hsa_restore_blocks",
    "hsa_block_resident",
    "hsa_select_blocks_noalloc",
    "hsa_forward",
    "hsa_get_info", "hsa_rewind", "hsa_state_layout", "hsa_workspace_layout", "hsa_set_wait_limit_ns",
    "hsa_device_status", "hsa_safe_pass_tiles",
    "hsa_last_cuda_error",
    "hsa_destroy", "hsa_status_string",
]


class hsa_config(C.Structure):
    _fields_ = [("num_heads", C.c_int32), ("head_dim", C.c_int32), ("page_tokens", C.c_int32),
                ("max_pages", C.c_int32), ("max_q_tokens", C.c_int32), ("max_topk", C.c_int32),
                ("lin_mode", C.c_int32), ("gate_act", C.c_int32), ("softmax_scale", C.c_float),
                ("flags", C.c_uint32), ("lin_rank", C.c_int32), ("lin_seg_tokens", C.c_int32),
                ("split_blocks", C.c_int32), ("feature_map", C.c_int32)]


class hsa_select_opts(C.Structure):
    _fields_ = [("inter_block_pages", C.c_int32), ("intra_first_page", C.c_int32),
                ("intra_budgets_dev", C.c_void_p), ("kv_pages_dev", C.c_void_p), ("n_kv_pages", C.c_int32),
                ("kv_page_blocks", C.c_int32)]


class hsa_sizes(C.Structure):
    _fields_ = [("k_pool", C.c_size_t), ("v_pool", C.c_size_t), ("state", C.c_size_t),
                ("workspace", C.c_size_t), ("kc_pool", C.c_size_t), ("vc_pool", C.c_size_t)]


class hsa_buffers(C.Structure):
    _fields_ = [("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("state", C.c_void_p),
                ("workspace", C.c_void_p), ("kc_pool", C.c_void_p), ("vc_pool", C.c_void_p),
                ("e_k", C.c_void_p), ("e_v", C.c_void_p)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} not found: build it with `python -m paper_2609_34606_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, u32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32
    lib.hsa_query_sizes.argtypes = [C.POINTER(hsa_config), C.POINTER(hsa_sizes)]
    lib.hsa_create.argtypes = [C.POINTER(vp), C.POINTER(hsa_config), C.POINTER(hsa_buffers), vp]
    lib.hsa_append_kv.argtypes = [vp, vp, vp, i32, i64, i64, vp]
    lib.hsa_select_blocks.argtypes = [vp, vp, i32, i64, i64, i64, i32, vp, i32, vp, vp, vp]
    lib.hsa_select_blocks_ex.argtypes = [vp, vp, i32, i64, i64, i64, i32, vp, i32, C.POINTER(hsa_select_opts), vp, vp,
                                         vp]
    lib.hsa_retrieve_kv_pages.argtypes = [vp, vp, i32, i64, i64, i32, i32, vp, vp, C.POINTER(i32), vp]
    lib.hsa_evict_blocks.argtypes = [vp, i32, i32, vp, vp, vp]
    lib.hsa_restore_blocks.argtypes = [vp, i32, i32, vp, vp, vp]
    lib.hsa_block_resident.argtypes = [vp, i32, C.POINTER(i32)]
    lib.hsa_select_blocks_adaptive.argtypes = [vp, vp, i32, i64, i64, i64, i32, C.c_float, C.c_float, i32, vp, vp,
                                               vp, vp]
    lib.hsa_select_blocks_noalloc.argtypes = [vp, i32, i64, i64, i32, i32, vp, i32, i64, i64, i32, C.c_float,
                                              vp, i32, vp, vp, vp, vp]
    lib.hsa_forward.argtypes = [vp, vp, i32, i64, i64, i64, i32, vp, vp, i32, vp, vp, i64, i64, i64,
                                vp, i64, i64, u32, vp]
    lib.hsa_get_info.argtypes = [vp, C.POINTER(i64), C.POINTER(i32)]
    lib.hsa_rewind.argtypes = [vp, i64]
    lib.hsa_state_layout.argtypes = [vp, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t),
                                     C.POINTER(C.c_size_t)]
    lib.hsa_workspace_layout.argtypes = [vp, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    lib.hsa_set_wait_limit_ns.argtypes = [vp, C.c_uint64]
    lib.hsa_device_status.argtypes = [vp, C.POINTER(i32)]
    lib.hsa_safe_pass_tiles.argtypes = [vp, C.POINTER(i64)]
    lib.hsa_last_cuda_error.argtypes = [vp]
    lib.hsa_destroy.argtypes = [vp]
    lib.hsa_status_string.argtypes = [C.c_int]
    lib.hsa_status_string.restype = C.c_char_p
    for name in EXPORTS:
        if name != "hsa_status_string":
            getattr(lib, name).restype = C.c_int
    return lib


_lib = _load()


class HSAError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {hsa_status_string(code)} ({code})")


def hsa_status_string(code: int) -> str:
    return _lib.hsa_status_string(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != HSA_OK:
        raise HSAError(code, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _thd(t: torch.Tensor, name: str) -> Tuple[int, int]:
    """(token stride, head stride) in elements of a bf16 [tokens, H, d] tensor, dim stride 1."""
    if t.dtype != torch.bfloat16 or t.dim() != 3 or not t.is_cuda or t.stride(2) != 1:
        raise ValueError(f"{name}: expected a CUDA bf16 [tokens, H, d] tensor with unit dim stride")
    return t.stride(0), t.stride(1)


# ------------------------------------------------------------------ C-named functions
def hsa_query_sizes(cfg: hsa_config) -> hsa_sizes:
    out = hsa_sizes()
    _check(_lib.hsa_query_sizes(C.byref(cfg), C.byref(out)), "hsa_query_sizes")
    return out


def hsa_create(cfg: hsa_config, bufs: hsa_buffers, page_alloc_order: Optional[torch.Tensor]) -> int:
    handle = C.c_void_p()
    order_ptr = None
    if page_alloc_order is not None:
        order = page_alloc_order.to(device="cpu", dtype=torch.int32).contiguous()
        order_ptr = order.data_ptr()
    _check(_lib.hsa_create(C.byref(handle), C.byref(cfg), C.byref(bufs), order_ptr), "hsa_create")
    return handle.value


def hsa_append_kv(ctx: int, k: torch.Tensor, v: torch.Tensor) -> None:
    ts, hs = _thd(k, "k")
    if _thd(v, "v") != (ts, hs) or v.shape != k.shape:
        raise ValueError("k and v must share shape and strides")
    _check(_lib.hsa_append_kv(ctx, k.data_ptr(), v.data_ptr(), k.shape[0], ts, hs, _stream()),
           "hsa_append_kv")


def hsa_select_blocks(ctx: int, q: torch.Tensor, q_pos0: int, causal: bool, budgets: torch.Tensor,
                      q_group_tokens: int, sel_idx: torch.Tensor, sel_cnt: torch.Tensor) -> None:
    ts, hs = _thd(q, "q")
    _check(_lib.hsa_select_blocks(ctx, q.data_ptr(), q.shape[0], ts, hs, int(q_pos0), int(causal),
                                  budgets.data_ptr(), int(q_group_tokens), sel_idx.data_ptr(),
                                  sel_cnt.data_ptr(), _stream()), "hsa_select_blocks")


def hsa_select_blocks_ex(ctx: int, q: torch.Tensor, q_pos0: int, causal: bool, budgets: torch.Tensor,
                         q_group_tokens: int, inter_block_pages: int, intra_first_page: int,
                         intra_budgets: Optional[torch.Tensor], sel_idx: torch.Tensor, sel_cnt: torch.Tensor,
                         kv_pages: Optional[torch.Tensor] = None, kv_page_blocks: int = 0) -> None:
    ts, hs = _thd(q, "q")
    opts = hsa_select_opts(int(inter_block_pages), int(intra_first_page), _ptr(intra_budgets), _ptr(kv_pages),
                           0 if kv_pages is None else int(kv_pages.numel()), int(kv_page_blocks))
    _check(_lib.hsa_select_blocks_ex(ctx, q.data_ptr(), q.shape[0], ts, hs, int(q_pos0), int(causal),
                                     budgets.data_ptr(), int(q_group_tokens), C.byref(opts), sel_idx.data_ptr(),
                                     sel_cnt.data_ptr(), _stream()), "hsa_select_blocks_ex")


def hsa_retrieve_kv_pages(ctx: int, q: torch.Tensor, kv_page_blocks: int, top_kp: int, page_ids: torch.Tensor,
                          scores: Optional[torch.Tensor] = None) -> int:
    """Returns the number of ids written to page_ids (int32, device)."""
    ts, hs = _thd(q, "q")
    n = C.c_int32(0)
    _check(_lib.hsa_retrieve_kv_pages(ctx, q.data_ptr(), q.shape[0], ts, hs, int(kv_page_blocks), int(top_kp),
                                      page_ids.data_ptr(), _ptr(scores), C.byref(n), _stream()),
           "hsa_retrieve_kv_pages")
    return n.value


def hsa_evict_blocks(ctx: int, first_block: int, n_blocks: int, host_k: torch.Tensor, host_v: torch.Tensor) -> None:
    _check(_lib.hsa_evict_blocks(ctx, int(first_block), int(n_blocks), host_k.data_ptr(), host_v.data_ptr(),
                                 _stream()), "hsa_evict_blocks")


def hsa_restore_blocks(ctx: int, first_block: int, n_blocks: int, host_k: torch.Tensor, host_v: torch.Tensor) -> None:
    _check(_lib.hsa_restore_blocks(ctx, int(first_block), int(n_blocks), host_k.data_ptr(), host_v.data_ptr(),
                                   _stream()), "hsa_restore_blocks")


def hsa_block_resident(ctx: int, block: int) -> bool:
    r = C.c_int32(0)
    _check(_lib.hsa_block_resident(ctx, int(block), C.byref(r)), "hsa_block_resident")
    return bool(r.value)


def hsa_select_blocks_adaptive(ctx: int, q: torch.Tensor, q_pos0: int, causal: bool, tau_min: float,
                               tau_max: float, q_group_tokens: int, sel_idx: torch.Tensor,
                               sel_cnt: torch.Tensor, gini_tau: Optional[torch.Tensor] = None) -> None:
    ts, hs = _thd(q, "q")
    _check(_lib.hsa_select_blocks_adaptive(ctx, q.data_ptr(), q.shape[0], ts, hs, int(q_pos0), int(causal),
                                           float(tau_min), float(tau_max), int(q_group_tokens),
                                           sel_idx.data_ptr(), sel_cnt.data_ptr(), _ptr(gini_tau), _stream()),
           "hsa_select_blocks_adaptive")


def hsa_select_blocks_noalloc(q: torch.Tensor, ksum: torch.Tensor, n_tokens: int, q_pos0: int, causal: bool,
                              softmax_scale: float, budgets: torch.Tensor, sel_idx: torch.Tensor,
                              sel_cnt: torch.Tensor, status: Optional[torch.Tensor] = None) -> None:
    """Allocation-free selection: ksum is the fp32 [H, blocks, d] key-sum view of a context's state
    (or any tensor of that layout); sel_idx is int32 [H, 1, max_topk], sel_cnt int32 [H, 1]."""
    ts, hs = _thd(q, "q")
    if ksum.dtype != torch.float32 or ksum.dim() != 3 or not ksum.is_contiguous():
        raise ValueError("ksum: expected a contiguous CUDA fp32 [H, blocks, d] tensor")
    _check(_lib.hsa_select_blocks_noalloc(q.data_ptr(), q.shape[0], ts, hs, q.shape[1], q.shape[2],
                                          ksum.data_ptr(), ksum.shape[1], int(n_tokens), int(q_pos0),
                                          int(causal), float(softmax_scale), budgets.data_ptr(),
                                          sel_idx.shape[-1], sel_idx.data_ptr(), sel_cnt.data_ptr(),
                                          _ptr(status), _stream()), "hsa_select_blocks_noalloc")


def hsa_forward(ctx: int, q: torch.Tensor, q_pos0: int, causal: bool, sel_idx: Optional[torch.Tensor],
                sel_cnt: Optional[torch.Tensor], q_group_tokens: int, g_lin: Optional[torch.Tensor],
                g_sp: Optional[torch.Tensor], out: torch.Tensor, flags: int = 0) -> None:
    ts, hs = _thd(q, "q")
    ots, ohs = _thd(out, "out")
    gts = ghs = gds = 0
    for g in (g_lin, g_sp):
        if g is not None:
            if g.dtype != torch.bfloat16 or not g.is_cuda or g.dim() not in (2, 3):
                raise ValueError("gates: expected CUDA bf16 [tokens, H] or [tokens, H, d]")
            s = (g.stride(0), g.stride(1), g.stride(2) if g.dim() == 3 else 0)
            if (gts, ghs, gds) != (0, 0, 0) and (gts, ghs, gds) != s:
                raise ValueError("g_lin and g_sp must share strides")
            gts, ghs, gds = s
    _check(_lib.hsa_forward(ctx, q.data_ptr(), q.shape[0], ts, hs, int(q_pos0), int(causal),
                            _ptr(sel_idx), _ptr(sel_cnt), int(q_group_tokens), _ptr(g_lin), _ptr(g_sp),
                            gts, ghs, gds, out.data_ptr(), ots, ohs, int(flags), _stream()),
           "hsa_forward")


def hsa_get_info(ctx: int) -> Tuple[int, int]:
    n, b = C.c_int64(), C.c_int32()
    _check(_lib.hsa_get_info(ctx, C.byref(n), C.byref(b)), "hsa_get_info")
    return n.value, b.value


def hsa_rewind(ctx: int, n_tokens: int) -> None:
    _check(_lib.hsa_rewind(ctx, int(n_tokens)), "hsa_rewind")


def hsa_state_layout(ctx: int) -> Tuple[int, int, int]:
    a, b, c = C.c_size_t(), C.c_size_t(), C.c_size_t()
    _check(_lib.hsa_state_layout(ctx, C.byref(a), C.byref(b), C.byref(c)), "hsa_state_layout")
    return a.value, b.value, c.value


def hsa_workspace_layout(ctx: int) -> Tuple[int, int]:
    a, b = C.c_size_t(), C.c_size_t()
    _check(_lib.hsa_workspace_layout(ctx, C.byref(a), C.byref(b)), "hsa_workspace_layout")
    return a.value, b.value


def hsa_set_wait_limit_ns(ctx: int, wait_ns: int) -> None:
    _check(_lib.hsa_set_wait_limit_ns(ctx, int(wait_ns)), "hsa_set_wait_limit_ns")


def hsa_device_status(ctx: int) -> int:
    s = C.c_int32()
    _check(_lib.hsa_device_status(ctx, C.byref(s)), "hsa_device_status")
    return s.value


def hsa_safe_pass_tiles(ctx: int) -> int:
    n = C.c_int64()
    _check(_lib.hsa_safe_pass_tiles(ctx, C.byref(n)), "hsa_safe_pass_tiles")
    return n.value


def hsa_last_cuda_error(ctx: int) -> int:
    return _lib.hsa_last_cuda_error(ctx)


def hsa_destroy(ctx: int) -> None:
    _check(_lib.hsa_destroy(ctx), "hsa_destroy")


# ------------------------------------------------------------------ convenience wrapper
class HSAContext:
    """One attention layer of one sequence: allocates the caller-owned buffers with torch and
    forwards every operation to the C ABI."""

    def __init__(self, H: int, d: int, max_pages: int, max_q_tokens: int, max_topk: int,
                 lin_mode: int = HSA_LIN_STATE, gate_act: int = 0, softmax_scale: float = 0.0,
                 causal: bool = False, page_order: Optional[torch.Tensor] = None,
                 device: str | torch.device = "cuda:0", adaptive: bool = False, lin_rank: int = 0, lin_seg_tokens: int = 0,
                 e_k: Optional[torch.Tensor] = None, e_v: Optional[torch.Tensor] = None, split_blocks: int = 0,
                 grid_barrier_select: bool = False, feature_map: int = 0):
        self.device = torch.device(device)
        self.H, self.d = H, d
        self.max_pages, self.max_q_tokens, self.max_topk = max_pages, max_q_tokens, max_topk
        self.cfg = hsa_config(H, d, PAGE_TOKENS, max_pages, max_q_tokens, max_topk, lin_mode, gate_act,
                              softmax_scale, (HSA_CFG_CAUSAL if causal else 0) | (HSA_CFG_ADAPTIVE if adaptive else 0) |
                              (HSA_CFG_GRID_BARRIER_SELECT if grid_barrier_select else 0),
                              lin_rank, lin_seg_tokens, split_blocks, feature_map)
        self.sizes = hsa_query_sizes(self.cfg)
        with torch.cuda.device(self.device):
            mk = lambda n: torch.empty(max(n, 16), dtype=torch.uint8, device=self.device)
            self.k_pool, self.v_pool = mk(self.sizes.k_pool), mk(self.sizes.v_pool)
            self.state, self.workspace = mk(self.sizes.state), mk(self.sizes.workspace)
            self.kc_pool = mk(self.sizes.kc_pool) if self.sizes.kc_pool else None
            self.vc_pool = mk(self.sizes.vc_pool) if self.sizes.vc_pool else None
            self.e_k, self.e_v = e_k, e_v   # keep the projection weights alive
            bufs = hsa_buffers(self.k_pool.data_ptr(), self.v_pool.data_ptr(), self.state.data_ptr(),
                               self.workspace.data_ptr(), _ptr(self.kc_pool), _ptr(self.vc_pool),
                               _ptr(e_k), _ptr(e_v))
            self.ctx = hsa_create(self.cfg, bufs, page_order)
        self._off_ksum = hsa_state_layout(self.ctx)[2]

    # -- state views (fp32) for tests and snapshots
    def _view(self, off: int, shape) -> torch.Tensor:
        n = 1
        for s in shape:
            n *= s
        return self.state[off:off + 4 * n].view(torch.float32).view(*shape)

    @property
    def S(self) -> torch.Tensor:
        # (the state lives in two slots that take turns: ask where the current one is)
        return self._view(hsa_state_layout(self.ctx)[0], (self.H, self.d, self.d))

    @property
    def z(self) -> torch.Tensor:
        return self._view(hsa_state_layout(self.ctx)[1], (self.H, self.d))

    @property
    def ksum(self) -> torch.Tensor:
        return self._view(self._off_ksum, (self.H, self.max_pages, self.d))

    @property
    def n_tokens(self) -> int:
        return hsa_get_info(self.ctx)[0]

    @property
    def n_blocks(self) -> int:
        return hsa_get_info(self.ctx)[1]

    def n_groups(self, n_q: int, group_tokens: int) -> int:
        return (n_q + group_tokens - 1) // group_tokens if group_tokens > 0 else 1

    def append_kv(self, k: torch.Tensor, v: torch.Tensor) -> None:
        hsa_append_kv(self.ctx, k, v)

    def alloc_selection(self, n_q: int, group_tokens: int = 0):
        g = self.n_groups(n_q, group_tokens)
        return (torch.zeros(self.H, g, self.max_topk, dtype=torch.int32, device=self.device),
                torch.zeros(self.H, g, dtype=torch.int32, device=self.device))

    def select_blocks(self, q: torch.Tensor, budgets: torch.Tensor, q_pos0: Optional[int] = None,
                      causal: bool = False, group_tokens: int = 0, sel=None):
        q_pos0 = self.n_tokens if q_pos0 is None else q_pos0
        sel_idx, sel_cnt = sel if sel is not None else self.alloc_selection(q.shape[0], group_tokens)
        hsa_select_blocks(self.ctx, q, q_pos0, causal, budgets, group_tokens, sel_idx, sel_cnt)
        return sel_idx, sel_cnt

    def select_blocks_ex(self, q: torch.Tensor, budgets: torch.Tensor, inter_block_pages: int = 2,
                         intra_first_page: int = -1, intra_budgets: Optional[torch.Tensor] = None,
                         q_pos0: Optional[int] = None, causal: bool = False, group_tokens: int = 0, sel=None,
                         kv_pages: Optional[torch.Tensor] = None, kv_page_blocks: int = 0):
        """Selection with coarse inter-chunk blocks (runs of inter_block_pages pages) and single-page
        intra-chunk blocks from intra_first_page on, optionally restricted to the retrieved KV pages
        (see hsa_select_blocks_ex)."""
        q_pos0 = self.n_tokens if q_pos0 is None else q_pos0
        sel_idx, sel_cnt = sel if sel is not None else self.alloc_selection(q.shape[0], group_tokens)
        hsa_select_blocks_ex(self.ctx, q, q_pos0, causal, budgets, group_tokens, inter_block_pages,
                             intra_first_page, intra_budgets, sel_idx, sel_cnt, kv_pages, kv_page_blocks)
        return sel_idx, sel_cnt

    def retrieve_kv_pages(self, q: torch.Tensor, kv_page_blocks: int, top_kp: int = 4, with_scores: bool = False):
        """Stage-2 page retrieval: (int32 ids of the kept KV pages, ascending[, fp32 score of every page])."""
        n_pages = (self.n_blocks + kv_page_blocks - 1) // kv_page_blocks
        ids = torch.zeros(max(1, min(top_kp, n_pages)), dtype=torch.int32, device=self.device)
        scores = torch.zeros(max(1, n_pages), dtype=torch.float32, device=self.device) if with_scores else None
        n = hsa_retrieve_kv_pages(self.ctx, q, kv_page_blocks, top_kp, ids, scores)
        return (ids[:n], scores[:n_pages]) if with_scores else ids[:n]

    def evict_blocks(self, first_block: int, n_blocks: int):
        """Moves the K / V tiles of the blocks to pinned host memory; returns the two host tensors."""
        shape = (n_blocks, self.H, PAGE_TOKENS, self.d)
        hk = torch.empty(shape, dtype=torch.bfloat16).pin_memory()
        hv = torch.empty(shape, dtype=torch.bfloat16).pin_memory()
        hsa_evict_blocks(self.ctx, first_block, n_blocks, hk, hv)
        return hk, hv

    def restore_blocks(self, first_block: int, host_k: torch.Tensor, host_v: torch.Tensor) -> None:
        hsa_restore_blocks(self.ctx, first_block, host_k.shape[0], host_k, host_v)

    def block_resident(self, block: int) -> bool:
        return hsa_block_resident(self.ctx, block)

    def select_blocks_adaptive(self, q: torch.Tensor, tau_min: float, tau_max: float,
                               q_pos0: Optional[int] = None, causal: bool = False, group_tokens: int = 0):
        """Cumulative-mass selection with the Gini threshold map; returns (sel_idx, sel_cnt, gini_tau)
        with gini_tau fp32 [2, H] = (Gini, threshold) per head."""
        q_pos0 = self.n_tokens if q_pos0 is None else q_pos0
        sel_idx, sel_cnt = self.alloc_selection(q.shape[0], group_tokens)
        gt = torch.zeros(2, self.H, dtype=torch.float32, device=self.device)
        hsa_select_blocks_adaptive(self.ctx, q, q_pos0, causal, tau_min, tau_max, group_tokens, sel_idx, sel_cnt, gt)
        return sel_idx, sel_cnt, gt

    def forward(self, q: torch.Tensor, sel_idx, sel_cnt, q_pos0: Optional[int] = None,
                causal: bool = False, group_tokens: int = 0, g_lin=None, g_sp=None, flags: int = 0,
                out: Optional[torch.Tensor] = None) -> torch.Tensor:
        q_pos0 = self.n_tokens if q_pos0 is None else q_pos0
        if out is None:
            out = torch.empty(q.shape, dtype=torch.bfloat16, device=self.device)
        hsa_forward(self.ctx, q, q_pos0, causal, sel_idx, sel_cnt, group_tokens, g_lin, g_sp, out, flags)
        return out

    def rewind(self, n_tokens: int) -> None:
        hsa_rewind(self.ctx, n_tokens)

    def device_status(self) -> int:
        return hsa_device_status(self.ctx)

    def set_wait_limit_ns(self, wait_ns: int) -> None:
        hsa_set_wait_limit_ns(self.ctx, wait_ns)

    def barrier_words(self) -> torch.Tensor:
        """uint32-as-int32 view [2] of the selection kernel's grid barrier {arrive count, generation}."""
        off = hsa_workspace_layout(self.ctx)[1]
        return self.workspace[off:off + 8].view(torch.int32)

    def safe_pass_tiles(self) -> int:
        return hsa_safe_pass_tiles(self.ctx)

    def destroy(self) -> None:
        if getattr(self, "ctx", None):
            hsa_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
