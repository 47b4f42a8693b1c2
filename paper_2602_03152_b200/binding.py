"""Thin ctypes binding of `libfasa.so`, the C-ABI CUDA library (include/fasa.h).

Argument marshalling only: every step of the decode path runs in the library's
kernels.  Tensors are torch CUDA tensors used as device memory; their data
pointers are passed through unchanged.  There is no CPU fallback: if the shared
object is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libfasa.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
DEV_LEN_CLAMPED, DEV_APPEND_FULL, DEV_IDX_CLAMPED, DEV_NSEL_CLAMPED, DEV_PAGE_CLAMPED, DEV_TIMEOUT = 1, 2, 4, 8, 16, 32

# Every entry point include/fasa.h declares.
SYMBOLS = [
    "fasa_create", "fasa_destroy", "fasa_proxy_row_elems", "fasa_workspace_bytes",
    "fasa_status_string", "fasa_last_cuda_error", "fasa_get_device_status", "fasa_launch_count",
    "fasa_kv_append", "fasa_proxy_build", "fasa_fc_score", "fasa_topk", "fasa_sparse_decode_attn",
    "fasa_full_decode_attn", "fasa_decode_step", "fasa_stage_bytes", "fasa_decode_step_host",
    "fasa_sparse_decode_attn_static", "fasa_set_step_mode", "fasa_step_cluster_size",
    "fasa_append_decode_step", "fasa_proxy_bytes", "fasa_select_step",
    "fasa_m_nondom_row_elems", "fasa_m_split", "fasa_m_kv_append", "fasa_m_sparse_decode_attn", "fasa_m_decode_step",
    "fasa_m_resident_bytes", "fasa_m_set_resident", "fasa_m_resident_build",
    "fasa_fc_score_batched", "fasa_topk_batched", "fasa_sparse_decode_attn_batched", "fasa_decode_step_batched",
    "fasa_calib_workspace_bytes", "fasa_calib_accumulate", "fasa_calib_select", "fasa_set_block_table",
]


class FasaError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: status {status} ({detail})")


class FasaConfig(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("max_len", ctypes.c_int32), ("n_dom", ctypes.c_int32),
        ("rope_pairing", ctypes.c_int32), ("group_reduce", ctypes.c_int32), ("select_heads", ctypes.c_int32),
        ("n_sink", ctypes.c_int32), ("n_recent", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
        ("k_stride_b", ctypes.c_int64), ("k_stride_h", ctypes.c_int64), ("k_stride_t", ctypes.c_int64),
        ("v_stride_b", ctypes.c_int64), ("v_stride_h", ctypes.c_int64), ("v_stride_t", ctypes.c_int64),
        ("page_size", ctypes.c_int32), ("n_pages", ctypes.c_int32),
    ]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libfasa.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2602_03152_b200.build`; "
            "the FASA decode path has no other implementation")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    sig = {
        "fasa_create": (i32, [ctypes.POINTER(FasaConfig), vp, ctypes.POINTER(vp)]),
        "fasa_destroy": (i32, [vp]),
        "fasa_proxy_row_elems": (i32, [i32]),
        "fasa_proxy_bytes": (i32, [vp, ctypes.POINTER(ctypes.c_size_t)]),
        "fasa_workspace_bytes": (i32, [vp, i32, ctypes.POINTER(ctypes.c_size_t)]),
        "fasa_status_string": (ctypes.c_char_p, [i32]),
        "fasa_last_cuda_error": (ctypes.c_char_p, [vp]),
        "fasa_get_device_status": (i32, [vp, vp, ctypes.POINTER(i32)]),
        "fasa_launch_count": (i64, [vp]),
        "fasa_kv_append": (i32, [vp] * 7 + [i32, vp]),
        "fasa_proxy_build": (i32, [vp] * 5),
        "fasa_fc_score": (i32, [vp] * 6),
        "fasa_topk": (i32, [vp, vp, vp, i32, i32, vp, vp, vp, vp]),
        "fasa_sparse_decode_attn": (i32, [vp] * 6 + [i32] + [vp] * 4),
        "fasa_full_decode_attn": (i32, [vp] * 9),
        "fasa_sparse_decode_attn_static": (i32, [vp] * 6 + [i32] + [vp] * 3),
        "fasa_decode_step": (i32, [vp] * 6 + [i32, i32] + [vp] * 7),
        "fasa_set_step_mode": (i32, [vp, i32]),
        "fasa_step_cluster_size": (i32, [vp]),
        "fasa_append_decode_step": (i32, [vp] * 8 + [i32, i32] + [vp] * 7),
        "fasa_select_step": (i32, [vp] * 8 + [i32, i32] + [vp] * 4),
        "fasa_m_nondom_row_elems": (i32, [i32]),
        "fasa_m_split": (i32, [vp] * 5),
        "fasa_m_kv_append": (i32, [vp] * 7 + [i32, vp]),
        "fasa_m_sparse_decode_attn": (i32, [vp] * 7 + [i32] + [vp] * 4),
        "fasa_m_decode_step": (i32, [vp] * 8 + [i32, i32] + [vp] * 7),
        "fasa_m_resident_bytes": (i64, [vp]),
        "fasa_m_set_resident": (i32, [vp, vp, vp]),
        "fasa_m_resident_build": (i32, [vp] * 6),
        "fasa_fc_score_batched": (i32, [vp, vp, vp, vp, i32, vp, vp]),
        "fasa_topk_batched": (i32, [vp, vp, vp, i32, i32, i32, vp, vp, vp]),
        "fasa_sparse_decode_attn_batched": (i32, [vp] * 6 + [i32, i32] + [vp] * 4),
        "fasa_decode_step_batched": (i32, [vp] * 6 + [i32, i32, i32] + [vp] * 7),
        "fasa_stage_bytes": (i32, [vp, ctypes.POINTER(ctypes.c_size_t)]),
        "fasa_decode_step_host": (i32, [vp] * 9 + [i32, i32] + [vp] * 7),
        "fasa_calib_workspace_bytes": (i32, [vp, i32, ctypes.POINTER(ctypes.c_size_t)]),
        "fasa_calib_accumulate": (i32, [vp, vp, vp, vp, i32, vp, vp, vp, vp]),
        "fasa_calib_select": (i32, [i32, i32, vp, vp, i32, i32, vp, vp]),
        "fasa_set_block_table": (i32, [vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _dp(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    """Device pointer of a contiguous CUDA tensor (None passes NULL)."""
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def proxy_row_elems(n_dom: int) -> int:
    return int(load_library().fasa_proxy_row_elems(n_dom))


class Fasa:
    """One context = one layer's configuration and dominant-FC table (fasa_create)."""

    def __init__(self, batch, n_q_heads, n_kv_heads, max_len, dom, *, head_dim=128, rope_pairing=0,
                 group_reduce=0, n_sink=0, n_recent=0, softmax_scale=0.0, k_strides=(0, 0, 0),
                 v_strides=(0, 0, 0), select_heads=0, page_size=0, n_pages=0):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        dom = torch.as_tensor(dom, dtype=torch.int32).contiguous().cpu()
        n_dom = dom.shape[-1] if dom.dim() == 2 else 0
        self.cfg = FasaConfig(batch, n_q_heads, n_kv_heads, head_dim, max_len, n_dom, rope_pairing,
                              group_reduce, select_heads, n_sink, n_recent, softmax_scale, *k_strides, *v_strides,
                              page_size, n_pages)
        if dom.dim() != 2 or dom.shape[0] != n_kv_heads:
            raise FasaError(ERR_INVALID_ARG, "fasa_create", "dom must be [n_kv_heads, n_dom]")
        st = self._lib.fasa_create(ctypes.byref(self.cfg), dom.data_ptr(), ctypes.byref(self._h))
        if st != OK:
            self._h = ctypes.c_void_p()
            raise FasaError(st, "fasa_create", self._lib.fasa_status_string(st).decode())
        self.batch, self.n_q_heads, self.n_kv_heads, self.max_len = batch, n_q_heads, n_kv_heads, max_len
        self.n_dom = n_dom
        self.page_size, self.n_pages = page_size, n_pages
        self._block_table = None
        group = n_q_heads // n_kv_heads
        self.select_heads = select_heads if select_heads > 0 else group    # query heads per index set
        self.n_sets = n_q_heads // self.select_heads                       # rows of scores / idx / n_sel per sequence
        self.row_elems = proxy_row_elems(n_dom)

    @classmethod
    def from_workload(cls, w, dom) -> "Fasa":
        return cls(w.batch, w.n_q_heads, w.n_kv_heads, w.max_len, dom, rope_pairing=w.pairing,
                   group_reduce=w.group_reduce, n_sink=w.n_sink, n_recent=w.n_recent, select_heads=w.sel_heads)

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.fasa_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int, where: str):
        if st != OK:
            detail = self._lib.fasa_status_string(st).decode()
            if st == ERR_CUDA:
                detail += ": " + self._lib.fasa_last_cuda_error(self._h).decode()
            raise FasaError(st, where, detail)

    # -- sizes ---------------------------------------------------------------
    def workspace_bytes(self, n_sel_max: int) -> int:
        out = ctypes.c_size_t()
        self._check(self._lib.fasa_workspace_bytes(self._h, n_sel_max, ctypes.byref(out)), "fasa_workspace_bytes")
        return int(out.value)

    def stage_bytes(self) -> int:
        out = ctypes.c_size_t()
        self._check(self._lib.fasa_stage_bytes(self._h, ctypes.byref(out)), "fasa_stage_bytes")
        return int(out.value)

    def set_step_mode(self, mode: int):
        """1: decode_step runs as one cluster kernel where available; 0: three separate calls; 2: as 1, with the
        one-CTA-per-row kernel behind topk."""
        self._check(self._lib.fasa_set_step_mode(self._h, mode), "fasa_set_step_mode")

    def step_cluster_size(self) -> int:
        return int(self._lib.fasa_step_cluster_size(self._h))

    def launch_count(self) -> int:
        return int(self._lib.fasa_launch_count(self._h))

    def device_status(self) -> int:
        out = ctypes.c_int32()
        self._check(self._lib.fasa_get_device_status(self._h, _stream(), ctypes.byref(out)), "fasa_get_device_status")
        return int(out.value)

    # -- device buffers (torch is the allocator) -------------------------------
    def proxy_bytes(self) -> int:
        out = ctypes.c_size_t()
        self._check(self._lib.fasa_proxy_bytes(self._h, ctypes.byref(out)), "fasa_proxy_bytes")
        return int(out.value)

    def alloc_proxy(self, device="cuda") -> torch.Tensor:
        """Zero-filled proxy-K buffer: [batch, kv heads, tiles of 16 tokens, 16 * row_elems] bf16
        (opaque tile-internal order, see include/fasa.h)."""
        tiles = (self.max_len + 15) // 16
        shape = (self.n_pages, self.n_kv_heads, self.page_size // 16) if self.page_size else (self.batch, self.n_kv_heads, tiles)
        t = torch.zeros(shape + (16 * self.row_elems,), dtype=torch.bfloat16, device=device)
        assert t.numel() * 2 == self.proxy_bytes()
        return t

    def alloc_workspace(self, n_sel_max: int, device="cuda") -> torch.Tensor:
        return torch.empty(self.workspace_bytes(n_sel_max), dtype=torch.uint8, device=device)

    def set_block_table(self, table: torch.Tensor):
        """Paged caches: int32 CUDA tensor [batch, ceil(max_len / page_size)] of physical pages.
        Kept by reference: its contents may change between calls."""
        self._check(self._lib.fasa_set_block_table(self._h, _dp(table, torch.int32)), "fasa_set_block_table")
        self._block_table = table

    def alloc_paged_cache(self, device="cuda") -> torch.Tensor:
        """A K or V page pool [n_pages, n_kv_heads, page_size, 128] (bf16)."""
        return torch.zeros((self.n_pages, self.n_kv_heads, self.page_size, 128), dtype=torch.bfloat16, device=device)

    def alloc_host_cache(self) -> torch.Tensor:
        """A K or V cache [batch, n_kv_heads, max_len, 128] (bf16) in page-locked host memory
        that the kernels address directly: the cache placement of FASA-M (Algorithm 2).  Pass it
        wherever a call takes k_cache / v_cache."""
        return torch.zeros((self.batch, self.n_kv_heads, self.max_len, 128), dtype=torch.bfloat16).pin_memory()

    # -- the calls of include/fasa.h --------------------------------------------
    def kv_append(self, k_cache, v_cache, proxy_k, seq_lens, k_new, v_new):
        n_new = k_new.shape[2]
        self._check(self._lib.fasa_kv_append(self._h, k_cache.data_ptr(), v_cache.data_ptr(), _dp(proxy_k),
                                             _dp(seq_lens, torch.int32), _dp(k_new, torch.bfloat16),
                                             _dp(v_new, torch.bfloat16), n_new, _stream()), "fasa_kv_append")

    def proxy_build(self, k_cache, proxy_k, seq_lens):
        self._check(self._lib.fasa_proxy_build(self._h, k_cache.data_ptr(), _dp(proxy_k),
                                               _dp(seq_lens, torch.int32), _stream()), "fasa_proxy_build")

    def fc_score(self, q, proxy_k, seq_lens, scores):
        self._check(self._lib.fasa_fc_score(self._h, _dp(q, torch.bfloat16), _dp(proxy_k),
                                            _dp(seq_lens, torch.int32), _dp(scores, torch.float32), _stream()),
                    "fasa_fc_score")

    def topk(self, scores, seq_lens, budget, idx, n_sel, workspace=None):
        n_sel_max = idx.shape[-1]
        self._check(self._lib.fasa_topk(self._h, _dp(scores, torch.float32), _dp(seq_lens, torch.int32), budget,
                                        n_sel_max, _dp(idx, torch.int32), _dp(n_sel, torch.int32), _dp(workspace),
                                        _stream()), "fasa_topk")

    def sparse_decode_attn(self, q, k_cache, v_cache, idx, n_sel, out, workspace, lse=None):
        n_sel_max = idx.shape[-1]
        self._check(self._lib.fasa_sparse_decode_attn(self._h, _dp(q, torch.bfloat16), k_cache.data_ptr(),
                                                      v_cache.data_ptr(), _dp(idx, torch.int32),
                                                      _dp(n_sel, torch.int32), n_sel_max, _dp(out, torch.float32),
                                                      _dp(lse), _dp(workspace), _stream()), "fasa_sparse_decode_attn")

    def sparse_decode_attn_static(self, q, k_cache, v_cache, idx, n_sel, out, lse=None):
        """fasa_sparse_decode_attn for callers that cannot provide a workspace: the split-K
        partials go to a fixed array inside the library (no allocation anywhere).  Calls share
        that array, so keep them ordered on one stream."""
        n_sel_max = idx.shape[-1]
        self._check(self._lib.fasa_sparse_decode_attn_static(
            self._h, _dp(q, torch.bfloat16), k_cache.data_ptr(), v_cache.data_ptr(), _dp(idx, torch.int32),
            _dp(n_sel, torch.int32), n_sel_max, _dp(out, torch.float32), _dp(lse), _stream()),
            "fasa_sparse_decode_attn_static")

    def full_decode_attn(self, q, k_cache, v_cache, seq_lens, out, workspace, lse=None):
        self._check(self._lib.fasa_full_decode_attn(self._h, _dp(q, torch.bfloat16), k_cache.data_ptr(),
                                                    v_cache.data_ptr(), _dp(seq_lens, torch.int32),
                                                    _dp(out, torch.float32), _dp(lse), _dp(workspace), _stream()),
                    "fasa_full_decode_attn")

    def decode_step(self, q, k_cache, v_cache, proxy_k, seq_lens, budget, scores, idx, n_sel, out, workspace=None,
                    lse=None):
        n_sel_max = idx.shape[-1]
        self._check(self._lib.fasa_decode_step(self._h, _dp(q, torch.bfloat16), k_cache.data_ptr(),
                                               v_cache.data_ptr(), _dp(proxy_k), _dp(seq_lens, torch.int32), budget,
                                               n_sel_max, _dp(scores, torch.float32), _dp(idx, torch.int32),
                                               _dp(n_sel, torch.int32), _dp(out, torch.float32), _dp(lse),
                                               _dp(workspace), _stream()), "fasa_decode_step")

    def append_decode_step(self, q, k_new, v_new, k_cache, v_cache, proxy_k, seq_lens, budget, scores, idx, n_sel,
                           out, workspace=None, lse=None):
        """Append one token per sequence, then the decode step on the grown cache (one launch in mode 1)."""
        n_sel_max = idx.shape[-1]
        self._check(self._lib.fasa_append_decode_step(
            self._h, _dp(q, torch.bfloat16), _dp(k_new, torch.bfloat16), _dp(v_new, torch.bfloat16),
            k_cache.data_ptr(), v_cache.data_ptr(), _dp(proxy_k), _dp(seq_lens, torch.int32), budget, n_sel_max,
            _dp(scores, torch.float32), _dp(idx, torch.int32), _dp(n_sel, torch.int32), _dp(out, torch.float32),
            _dp(lse), _dp(workspace), _stream()), "fasa_append_decode_step")

    def select_step(self, q, k_cache, v_cache, proxy_k, seq_lens, budget, scores, idx, n_sel, k_new=None, v_new=None):
        """Scoring and selection in one launch, no attention (appending form when k_new / v_new are given)."""
        n_sel_max = idx.shape[-1]
        self._check(self._lib.fasa_select_step(
            self._h, _dp(q, torch.bfloat16), _dp(k_new, torch.bfloat16), _dp(v_new, torch.bfloat16),
            k_cache.data_ptr(), v_cache.data_ptr(), _dp(proxy_k), _dp(seq_lens, torch.int32), budget, n_sel_max,
            _dp(scores, torch.float32), _dp(idx, torch.int32), _dp(n_sel, torch.int32), _stream()), "fasa_select_step")

    # -- memory-optimised variant with a split key cache (Algorithm 2) -----------------
    def alloc_host_nondom(self) -> torch.Tensor:
        """Page-locked host tensor [batch][n_kv_heads][max_len][128 - 2 n_dom] for the non-dominant key channels."""
        nd = int(self._lib.fasa_m_nondom_row_elems(self.n_dom))
        if nd == 0:
            raise FasaError(ERR_UNSUPPORTED, "fasa_m_nondom_row_elems", "n_dom must be a multiple of 4")
        t = torch.zeros((self.batch, self.n_kv_heads, self.max_len, nd), dtype=torch.bfloat16).pin_memory()
        return t

    def m_split(self, k_cache, k_nondom, seq_lens):
        self._check(self._lib.fasa_m_split(self._h, k_cache.data_ptr(), k_nondom.data_ptr(), _dp(seq_lens, torch.int32), _stream()),
                    "fasa_m_split")

    def m_kv_append(self, k_nondom, v_cache, proxy_k, seq_lens, k_new, v_new):
        self._check(self._lib.fasa_m_kv_append(self._h, k_nondom.data_ptr(), v_cache.data_ptr(), _dp(proxy_k), _dp(seq_lens, torch.int32),
                                               _dp(k_new, torch.bfloat16), _dp(v_new, torch.bfloat16), k_new.shape[2], _stream()),
                    "fasa_m_kv_append")

    def m_sparse_decode_attn(self, q, k_nondom, v_cache, proxy_k, idx, n_sel, out, workspace, lse=None):
        self._check(self._lib.fasa_m_sparse_decode_attn(self._h, _dp(q, torch.bfloat16), k_nondom.data_ptr(), v_cache.data_ptr(),
                                                        _dp(proxy_k), _dp(idx, torch.int32), _dp(n_sel, torch.int32), idx.shape[-1],
                                                        _dp(out, torch.float32), _dp(lse), _dp(workspace), _stream()),
                    "fasa_m_sparse_decode_attn")

    def m_decode_step(self, q, k_nondom, v_cache, proxy_k, seq_lens, budget, scores, idx, n_sel, out, workspace, lse=None,
                      k_new=None, v_new=None):
        self._check(self._lib.fasa_m_decode_step(
            self._h, _dp(q, torch.bfloat16), _dp(k_new, torch.bfloat16), _dp(v_new, torch.bfloat16), k_nondom.data_ptr(),
            v_cache.data_ptr(), _dp(proxy_k), _dp(seq_lens, torch.int32), budget, idx.shape[-1], _dp(scores, torch.float32),
            _dp(idx, torch.int32), _dp(n_sel, torch.int32), _dp(out, torch.float32), _dp(lse), _dp(workspace), _stream()),
            "fasa_m_decode_step")

    def alloc_resident(self) -> torch.Tensor:
        """Device buffer for the GPU-resident sink / recent rows of the memory-optimised variant, registered."""
        n = int(self._lib.fasa_m_resident_bytes(self._h))
        if n == 0:
            raise FasaError(ERR_UNSUPPORTED, "fasa_m_resident_bytes", "no forced positions, or no split key cache")
        buf = torch.empty(n, dtype=torch.uint8, device="cuda")
        self.m_set_resident(buf)
        return buf

    def m_set_resident(self, buf):
        self._check(self._lib.fasa_m_set_resident(self._h, None if buf is None else buf.data_ptr(), _stream()),
                    "fasa_m_set_resident")
        self._resident = buf                       # (kept by reference in the library)

    def m_resident_build(self, k_nondom, v_cache, proxy_k, seq_lens):
        self._check(self._lib.fasa_m_resident_build(self._h, k_nondom.data_ptr(), v_cache.data_ptr(), _dp(proxy_k),
                                                    _dp(seq_lens, torch.int32), _stream()), "fasa_m_resident_build")

    # -- blocks of query tokens: tensors carry a query axis after the batch axis ------
    def fc_score_batched(self, q, proxy_k, seq_lens, scores):
        self._check(self._lib.fasa_fc_score_batched(self._h, _dp(q, torch.bfloat16), _dp(proxy_k), _dp(seq_lens, torch.int32),
                                                    q.shape[1], _dp(scores, torch.float32), _stream()), "fasa_fc_score_batched")

    def topk_batched(self, scores, seq_lens, budget, idx, n_sel):
        self._check(self._lib.fasa_topk_batched(self._h, _dp(scores, torch.float32), _dp(seq_lens, torch.int32), scores.shape[1],
                                                budget, idx.shape[-1], _dp(idx, torch.int32), _dp(n_sel, torch.int32), _stream()),
                    "fasa_topk_batched")

    def sparse_decode_attn_batched(self, q, k_cache, v_cache, idx, n_sel, out, workspace, lse=None):
        self._check(self._lib.fasa_sparse_decode_attn_batched(
            self._h, _dp(q, torch.bfloat16), k_cache.data_ptr(), v_cache.data_ptr(), _dp(idx, torch.int32),
            _dp(n_sel, torch.int32), q.shape[1], idx.shape[-1], _dp(out, torch.float32), _dp(lse), _dp(workspace), _stream()),
            "fasa_sparse_decode_attn_batched")

    def decode_step_batched(self, q, k_cache, v_cache, proxy_k, seq_lens, budget, scores, idx, n_sel, out, workspace, lse=None):
        self._check(self._lib.fasa_decode_step_batched(
            self._h, _dp(q, torch.bfloat16), k_cache.data_ptr(), v_cache.data_ptr(), _dp(proxy_k), _dp(seq_lens, torch.int32),
            q.shape[1], budget, idx.shape[-1], _dp(scores, torch.float32), _dp(idx, torch.int32), _dp(n_sel, torch.int32),
            _dp(out, torch.float32), _dp(lse), _dp(workspace), _stream()), "fasa_decode_step_batched")

    # -- offline calibration (Algorithm 1) ---------------------------------------
    def calib_workspace_bytes(self, top_k: int) -> int:
        out = ctypes.c_size_t()
        self._check(self._lib.fasa_calib_workspace_bytes(self._h, top_k, ctypes.byref(out)), "fasa_calib_workspace_bytes")
        return int(out.value)

    def calib_accumulate(self, q, k_cache, seq_lens, top_k, ca_counts, n_used, workspace):
        """Adds this batch's top_k * CA sums (Eq. 4) to ca_counts [n_q_heads, 64] and the sample
        numbers to n_used [n_q_heads] (int64 CUDA tensors carried from call to call)."""
        self._check(self._lib.fasa_calib_accumulate(self._h, _dp(q, torch.bfloat16), k_cache.data_ptr(),
                                                    _dp(seq_lens, torch.int32), top_k, _dp(ca_counts, torch.int64),
                                                    _dp(n_used, torch.int64), _dp(workspace), _stream()),
                    "fasa_calib_accumulate")

    def decode_step_host(self, q_host, k_new_host, v_new_host, dev_stage, k_cache, v_cache, proxy_k, seq_lens,
                         budget, scores, idx, n_sel, out, out_host, workspace):
        """Host tensors in (pinned recommended), host tensor out; synchronises the stream."""
        for t in (q_host, k_new_host, v_new_host, out_host):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("host arguments must be contiguous CPU tensors")
        n_sel_max = idx.shape[-1]
        self._check(self._lib.fasa_decode_step_host(
            self._h, q_host.data_ptr(), k_new_host.data_ptr(), v_new_host.data_ptr(), _dp(dev_stage),
            k_cache.data_ptr(), v_cache.data_ptr(), _dp(proxy_k), _dp(seq_lens, torch.int32), budget, n_sel_max,
            _dp(scores, torch.float32), _dp(idx, torch.int32), _dp(n_sel, torch.int32), _dp(out, torch.float32),
            out_host.data_ptr(), _dp(workspace), _stream()), "fasa_decode_step_host")


def calib_select(ca_counts, n_used, n_kv_heads: int, top_k: int, n_dom: int):
    """Stage 2 of Algorithm 1 on the host: (I_dom int32 [n_kv_heads, n_dom] ascending, mean CA
    float64 [n_kv_heads, 64]) from the accumulated counts (any device; copied to the host)."""
    lib = load_library()
    counts = ca_counts.detach().to("cpu", torch.int64).contiguous()
    used = n_used.detach().to("cpu", torch.int64).contiguous()
    n_q_heads = counts.shape[0]
    dom = torch.zeros((n_kv_heads, n_dom), dtype=torch.int32)
    mean = torch.zeros((n_kv_heads, 64), dtype=torch.float64)
    st = lib.fasa_calib_select(n_q_heads, n_kv_heads, counts.data_ptr(), used.data_ptr(), top_k, n_dom,
                               dom.data_ptr(), mean.data_ptr())
    if st != OK:
        raise FasaError(st, "fasa_calib_select", lib.fasa_status_string(st).decode())
    return dom, mean
