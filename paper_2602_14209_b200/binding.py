"""Thin ctypes binding of ``libmage.so``: argument marshalling only.

Function names and arguments mirror ``include/mage.h``.  Tensors are torch CUDA
tensors (torch is used for device memory and streams, nothing else); every
step of the path runs inside the library's kernels.  There is no fallback: if
the library has not been built, the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmage.so")
_lib = None

MAGE_OK = 0
FLAG_SIMT_KERNELS = 1
FLAG_TEST_STALL = 2
DEV_BAD_INDEX, DEV_BAD_PAGE, DEV_TIMEOUT, DEV_CACHE_FULL = 1, 2, 4, 8


class MageError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


class mage_k8_t(ctypes.Structure):
    _fields_ = [("k8_cache", ctypes.c_void_p), ("k_scale", ctypes.c_void_p), ("scratch", ctypes.c_void_p)]


class mage_kv_t(ctypes.Structure):
    _fields_ = [
        ("P", ctypes.c_int32), ("H_q", ctypes.c_int32), ("H_kv", ctypes.c_int32), ("d", ctypes.c_int32),
        ("B", ctypes.c_int32), ("page_size", ctypes.c_int32),
        ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
        ("stride_p", ctypes.c_int64), ("stride_h", ctypes.c_int64), ("stride_n", ctypes.c_int64),
        ("block_table", ctypes.c_void_p), ("max_pages", ctypes.c_int32), ("num_pages", ctypes.c_int32),
        ("seq_lens", ctypes.c_void_p), ("N_max", ctypes.c_int32), ("flags", ctypes.c_int32),
    ]


EXPORTS = ("mage_pruned_workspace_bytes", "mage_exact_select_pruned", "mage_quest_workspace_bytes", "mage_quest_build", "mage_quest_select", "mage_append_block", "mage_workspace_bytes", "mage_exact_select", "mage_exact_select_events", "mage_exact_select_static", "mage_exact_attn", "mage_select_scores", "mage_topk", "mage_sparse_block_attn",
           "mage_k8_scratch_bytes", "mage_k8_quantize_cache", "mage_exact_select_k8", "mage_exact_select_k8_events", "mage_sparse_block_attn_k8",
           "mage_status_string", "mage_launch_count")


def load():
    """Load libmage.so (once).  Raises if it is missing: there is no other implementation to fall back to."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is not built; run `python -m paper_2602_14209_b200.build`")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint64
    lib.mage_workspace_bytes.restype = ctypes.c_size_t
    lib.mage_workspace_bytes.argtypes = [ctypes.POINTER(mage_kv_t), i32]
    lib.mage_exact_select.restype = ctypes.c_int
    lib.mage_exact_select.argtypes = [ctypes.POINTER(mage_kv_t), vp, vp, vp, ctypes.c_float, vp, vp, vp, ctypes.c_size_t, vp, vp]
    lib.mage_exact_select_events.restype = ctypes.c_int
    lib.mage_exact_select_events.argtypes = lib.mage_exact_select.argtypes + [ctypes.POINTER(ctypes.c_void_p)]
    lib.mage_exact_select_static.restype = ctypes.c_int
    lib.mage_exact_select_static.argtypes = [ctypes.POINTER(mage_kv_t), vp, vp, vp, ctypes.c_float, vp, vp, vp, vp]
    lib.mage_exact_attn.restype = ctypes.c_int
    lib.mage_exact_attn.argtypes = [ctypes.POINTER(mage_kv_t), vp, vp, vp, ctypes.c_float, vp, vp, ctypes.c_size_t, vp, vp]
    lib.mage_select_scores.restype = ctypes.c_int
    lib.mage_select_scores.argtypes = [ctypes.POINTER(mage_kv_t), vp, ctypes.c_float, vp, vp, ctypes.c_size_t, vp, vp]
    lib.mage_topk.restype = ctypes.c_int
    lib.mage_topk.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp, ctypes.c_size_t, vp]
    lib.mage_sparse_block_attn.restype = ctypes.c_int
    lib.mage_sparse_block_attn.argtypes = [ctypes.POINTER(mage_kv_t), vp, vp, vp, vp, vp, i32, ctypes.c_float, vp, vp, ctypes.c_size_t, vp, vp]
    lib.mage_append_block.restype = ctypes.c_int
    lib.mage_append_block.argtypes = [ctypes.POINTER(mage_kv_t), vp, vp, vp, vp, vp]
    lib.mage_pruned_workspace_bytes.restype = ctypes.c_size_t
    lib.mage_pruned_workspace_bytes.argtypes = [ctypes.POINTER(mage_kv_t), i32]
    lib.mage_exact_select_pruned.restype = ctypes.c_int
    lib.mage_exact_select_pruned.argtypes = [ctypes.POINTER(mage_kv_t), vp, vp, vp, ctypes.c_float, i32, ctypes.c_float, vp, vp, vp, vp, vp, vp,
                                             ctypes.c_size_t, vp, vp]
    lib.mage_quest_workspace_bytes.restype = ctypes.c_size_t
    lib.mage_quest_workspace_bytes.argtypes = [ctypes.POINTER(mage_kv_t), i32]
    lib.mage_quest_build.restype = ctypes.c_int
    lib.mage_quest_build.argtypes = [ctypes.POINTER(mage_kv_t), vp, vp, vp, vp]
    lib.mage_quest_select.restype = ctypes.c_int
    lib.mage_quest_select.argtypes = [ctypes.POINTER(mage_kv_t), vp, vp, vp, i32, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.mage_k8_scratch_bytes.restype = ctypes.c_size_t
    lib.mage_k8_scratch_bytes.argtypes = [ctypes.POINTER(mage_kv_t)]
    lib.mage_k8_quantize_cache.restype = ctypes.c_int
    lib.mage_k8_quantize_cache.argtypes = [ctypes.POINTER(mage_kv_t), i32, vp, vp, vp, vp]
    lib.mage_exact_select_k8.restype = ctypes.c_int
    lib.mage_exact_select_k8.argtypes = [ctypes.POINTER(mage_kv_t), ctypes.POINTER(mage_k8_t), vp, vp, vp, ctypes.c_float, vp, vp, vp,
                                         ctypes.c_size_t, vp, vp]
    lib.mage_exact_select_k8_events.restype = ctypes.c_int
    lib.mage_exact_select_k8_events.argtypes = lib.mage_exact_select_k8.argtypes + [ctypes.POINTER(ctypes.c_void_p)]
    lib.mage_sparse_block_attn_k8.restype = ctypes.c_int
    lib.mage_sparse_block_attn_k8.argtypes = [ctypes.POINTER(mage_kv_t), ctypes.POINTER(mage_k8_t), vp, vp, vp, vp, vp, i32, ctypes.c_float,
                                              vp, vp, ctypes.c_size_t, vp, vp]
    lib.mage_status_string.restype = ctypes.c_char_p
    lib.mage_status_string.argtypes = [ctypes.c_int]
    lib.mage_launch_count.restype = u64
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load().mage_status_string(int(code)).decode()


def launch_count() -> int:
    return int(load().mage_launch_count())


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


class KVCache:
    """Host-side description of the prefix KV cache of a batch of P problems (``mage_kv_t``).

    Contiguous: ``k``, ``v`` are [P, H_kv, N_max, d] bf16 views (any strides with d contiguous).
    Paged: ``k``, ``v`` are pools [num_pages, H_kv, page_size, d] and ``block_table`` is [P, max_pages] int32.
    ``seq_lens`` is a device int32 [P] tensor or None (every problem has N_max keys).
    The object only keeps references; it owns no memory of its own.
    """

    def __init__(self, k: torch.Tensor, v: torch.Tensor, H_q: int, B: int, seq_lens: Optional[torch.Tensor] = None,
                 block_table: Optional[torch.Tensor] = None, N_max: Optional[int] = None, flags: int = 0):
        assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.dim() == 4 and k.shape == v.shape
        assert k.stride() == v.stride() and k.stride(3) == 1
        self.k, self.v, self.seq_lens, self.block_table = k, v, seq_lens, block_table
        c = mage_kv_t()
        if block_table is None:
            P, H_kv, n, d = k.shape
            c.page_size = 0
            c.stride_p, c.stride_h, c.stride_n = k.stride(0), k.stride(1), k.stride(2)
            c.N_max = n if N_max is None else N_max
        else:
            assert k.is_contiguous() and v.is_contiguous() and block_table.dtype == torch.int32 and block_table.is_contiguous()
            num_pages, H_kv, page, d = k.shape
            P = block_table.shape[0]
            c.page_size, c.num_pages, c.max_pages = page, num_pages, block_table.shape[1]
            c.block_table = block_table.data_ptr()
            assert N_max is not None
            c.N_max = N_max
        c.P, c.H_q, c.H_kv, c.d, c.B, c.flags = P, H_q, H_kv, d, B, flags
        c.k_cache, c.v_cache = k.data_ptr(), v.data_ptr()
        if seq_lens is not None:
            assert seq_lens.dtype == torch.int32 and seq_lens.numel() == P and seq_lens.is_cuda
            c.seq_lens = seq_lens.data_ptr()
        self.c = c
        self.P, self.H_q, self.H_kv, self.d, self.B, self.N_max = P, H_q, H_kv, d, B, int(c.N_max)
        self.device = k.device

    def workspace_bytes(self, k_max: int = 1) -> int:
        return int(load().mage_workspace_bytes(ctypes.byref(self.c), int(k_max)))

    def new_workspace(self, k_max: int = 1) -> torch.Tensor:
        n = self.workspace_bytes(k_max)
        if n == 0:
            raise MageError(-1, "mage_workspace_bytes")
        return torch.empty(n, dtype=torch.uint8, device=self.device)


def mage_exact_select(kv: KVCache, q, k_blk, v_blk, sm_scale: float, out, scores, workspace, dev_status=None, stream=None,
                      events=None):
    """Step 1 of a block: exact attention into ``out`` and block scores into ``scores`` (see mage.h).

    ``events``: optional list of four recorded-on-demand ``torch.cuda.Event(enable_timing=True)`` objects; when given,
    the call goes through ``mage_exact_select_events`` and the library records them between its kernels.
    """
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    args = (ctypes.byref(kv.c), _ptr(q), _ptr(k_blk), _ptr(v_blk), float(sm_scale), _ptr(out), _ptr(scores), _ptr(workspace),
            ws_bytes, _ptr(dev_status), _stream(stream))
    if events is None:
        rc = load().mage_exact_select(*args)
    else:
        for e in events:                 # torch creates the CUDA event lazily, at its first record
            if not e.cuda_event:
                e.record()
        handles = (ctypes.c_void_p * 4)(*[ctypes.c_void_p(e.cuda_event) for e in events])
        rc = load().mage_exact_select_events(*args, handles)
    if rc != MAGE_OK:
        raise MageError(rc, "mage_exact_select")


def mage_exact_attn(kv: KVCache, q, k_blk, v_blk, sm_scale: float, out, workspace, dev_status=None, stream=None):
    """Exact attention of the block without the score pass (the main stream's half of Step 1; see mage.h)."""
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    rc = load().mage_exact_attn(ctypes.byref(kv.c), _ptr(q), _ptr(k_blk), _ptr(v_blk), float(sm_scale), _ptr(out), _ptr(workspace),
                                ws_bytes, _ptr(dev_status), _stream(stream))
    if rc != MAGE_OK:
        raise MageError(rc, "mage_exact_attn")


def mage_select_scores(kv: KVCache, q, sm_scale: float, scores, workspace, dev_status=None, stream=None):
    """Block scores from the queries and the cached keys alone (the select stream's own computation; see mage.h)."""
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    rc = load().mage_select_scores(ctypes.byref(kv.c), _ptr(q), float(sm_scale), _ptr(scores), _ptr(workspace), ws_bytes,
                                   _ptr(dev_status), _stream(stream))
    if rc != MAGE_OK:
        raise MageError(rc, "mage_select_scores")


STATIC_SCRATCH_BYTES = 32 << 20


def mage_exact_select_static(kv: KVCache, q, k_blk, v_blk, sm_scale: float, out, scores, dev_status=None, stream=None):
    """Step 1 without a caller workspace: the scratch is a fixed array inside the library (see mage.h).

    For hosts that may not allocate device memory when they call.  Descriptions that need more than
    STATIC_SCRATCH_BYTES are refused with MAGE_ERR_WORKSPACE.  Calls on one device share the scratch, so
    calls that could overlap on the GPU must be ordered by the caller.
    """
    rc = load().mage_exact_select_static(ctypes.byref(kv.c), _ptr(q), _ptr(k_blk), _ptr(v_blk), float(sm_scale), _ptr(out),
                                         _ptr(scores), _ptr(dev_status), _stream(stream))
    if rc != MAGE_OK:
        raise MageError(rc, "mage_exact_select_static")


def mage_topk(scores, seq_lens, P: int, H_kv: int, N_max: int, k: int, indices, k_eff, stream=None):
    """Per-KV-head Top-k of ``scores`` into ``indices`` / ``k_eff`` (see mage.h)."""
    rc = load().mage_topk(_ptr(scores), _ptr(seq_lens), P, H_kv, N_max, k, _ptr(indices), _ptr(k_eff), None, 0, _stream(stream))
    if rc != MAGE_OK:
        raise MageError(rc, "mage_topk")


def mage_sparse_block_attn(kv: KVCache, q, k_blk, v_blk, indices, k_eff, k: int, sm_scale: float, out, workspace=None,
                           dev_status=None, stream=None):
    """Reuse step: attention over the selected cache rows plus the block's own keys (see mage.h)."""
    rc = load().mage_sparse_block_attn(ctypes.byref(kv.c), _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(indices), _ptr(k_eff), int(k),
                                       float(sm_scale), _ptr(out), _ptr(workspace),
                                       workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                       _ptr(dev_status), _stream(stream))
    if rc != MAGE_OK:
        raise MageError(rc, "mage_sparse_block_attn")


class K8Keys:
    """The keys of a cache as e4m3 codes (``mage_k8_t``): ``codes`` is a uint8 tensor shaped and strided like ``kv.k``,
    ``k_scale`` is [P, H_kv] fp32, ``scratch`` the per-call buffer.  ``quantize`` fills codes (and, from row 0, the scales)."""

    def __init__(self, kv: KVCache):
        self.kv = kv
        self.codes = torch.empty_strided(kv.k.shape, kv.k.stride(), dtype=torch.uint8, device=kv.device)
        self.k_scale = torch.empty(kv.P, kv.H_kv, dtype=torch.float32, device=kv.device)
        n = int(load().mage_k8_scratch_bytes(ctypes.byref(kv.c)))
        if n == 0:
            raise MageError(-1, "mage_k8_scratch_bytes")
        self.scratch = torch.empty(n, dtype=torch.uint8, device=kv.device)
        self.c = mage_k8_t(self.codes.data_ptr(), self.k_scale.data_ptr(), self.scratch.data_ptr())

    def quantize(self, row_begin: int = 0, dev_status=None, stream=None):
        rc = load().mage_k8_quantize_cache(ctypes.byref(self.kv.c), int(row_begin), _ptr(self.codes), _ptr(self.k_scale), _ptr(dev_status),
                                           _stream(stream))
        if rc != MAGE_OK:
            raise MageError(rc, "mage_k8_quantize_cache")
        return self


def mage_exact_select_k8(kv: KVCache, k8: K8Keys, q, k_blk, v_blk, sm_scale: float, out, scores, workspace, dev_status=None, stream=None,
                         events=None):
    """mage_exact_select with the keys (and queries) in 8 bits (see mage.h); ``events`` as in ``mage_exact_select``."""
    args = (ctypes.byref(kv.c), ctypes.byref(k8.c), _ptr(q), _ptr(k_blk), _ptr(v_blk), float(sm_scale), _ptr(out), _ptr(scores),
            _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream(stream))
    if events is None:
        rc = load().mage_exact_select_k8(*args)
    else:
        for e in events:
            if not e.cuda_event:
                e.record()
        handles = (ctypes.c_void_p * 4)(*[ctypes.c_void_p(e.cuda_event) for e in events])
        rc = load().mage_exact_select_k8_events(*args, handles)
    if rc != MAGE_OK:
        raise MageError(rc, "mage_exact_select_k8")


def mage_sparse_block_attn_k8(kv: KVCache, k8: K8Keys, q, k_blk, v_blk, indices, k_eff, k: int, sm_scale: float, out, workspace=None,
                              dev_status=None, stream=None):
    """mage_sparse_block_attn with the keys (and queries) in 8 bits (see mage.h)."""
    rc = load().mage_sparse_block_attn_k8(ctypes.byref(kv.c), ctypes.byref(k8.c), _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(indices),
                                          _ptr(k_eff), int(k), float(sm_scale), _ptr(out), _ptr(workspace),
                                          workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                          _ptr(dev_status), _stream(stream))
    if rc != MAGE_OK:
        raise MageError(rc, "mage_sparse_block_attn_k8")


def mage_append_block(kv: KVCache, k_blk, v_blk, seq_lens, dev_status=None, stream=None):
    """End of a block: append the block's final K/V to the cache and add B to ``seq_lens`` (see mage.h)."""
    rc = load().mage_append_block(ctypes.byref(kv.c), _ptr(k_blk), _ptr(v_blk), _ptr(seq_lens), _ptr(dev_status), _stream(stream))
    if rc != MAGE_OK:
        raise MageError(rc, "mage_append_block")


QUEST_PAGE = 16


def mage_quest_build(kv: KVCache, page_min, page_max, dev_status=None, stream=None):
    """Quest-style page summaries (per-channel min / max of each whole 16-token page of the prefix; see mage.h)."""
    rc = load().mage_quest_build(ctypes.byref(kv.c), _ptr(page_min), _ptr(page_max), _ptr(dev_status), _stream(stream))
    if rc != MAGE_OK:
        raise MageError(rc, "mage_quest_build")


def mage_quest_select(kv: KVCache, q, page_min, page_max, k: int, page_scores, indices, k_eff, workspace, stream=None):
    """Per-block Quest-style selection: page scores, the k/16 best pages, their tokens as an index set (see mage.h)."""
    rc = load().mage_quest_select(ctypes.byref(kv.c), _ptr(q), _ptr(page_min), _ptr(page_max), int(k), _ptr(page_scores), _ptr(indices),
                                  _ptr(k_eff), _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream))
    if rc != MAGE_OK:
        raise MageError(rc, "mage_quest_select")


def quest_workspace(kv: KVCache, k: int) -> torch.Tensor:
    n = int(load().mage_quest_workspace_bytes(ctypes.byref(kv.c), int(k)))
    if n == 0:
        raise MageError(-1, "mage_quest_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=kv.device)


def pruned_workspace(kv: KVCache, k: int) -> torch.Tensor:
    n = int(load().mage_pruned_workspace_bytes(ctypes.byref(kv.c), int(k)))
    if n == 0:
        raise MageError(-1, "mage_pruned_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=kv.device)


def mage_exact_select_pruned(kv: KVCache, q, k_blk, v_blk, sm_scale: float, k: int, out, scores, indices, k_eff, workspace,
                             tiles_scored=None, dense_above: float = 0.5, dev_status=None, stream=None):
    """Step 1 + selection with the score pass restricted to the key tiles that can hold a selected key (see mage.h)."""
    rc = load().mage_exact_select_pruned(ctypes.byref(kv.c), _ptr(q), _ptr(k_blk), _ptr(v_blk), float(sm_scale), int(k), float(dense_above),
                                         _ptr(out), _ptr(scores), _ptr(indices), _ptr(k_eff), _ptr(tiles_scored), _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream(stream))
    if rc != MAGE_OK:
        raise MageError(rc, "mage_exact_select_pruned")

