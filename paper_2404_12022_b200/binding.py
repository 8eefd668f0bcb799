"""Python entry points of the C-ABI library, same names as in ``include/ht.h``.

Argument marshalling only: tensors are torch CUDA tensors whose ``data_ptr()`` goes
straight to the library, outputs are allocated with torch, work is enqueued on torch's
current stream.  Every step of the path runs in the library's kernels; there is no
fallback, and a missing ``libht.so`` raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libht.so")

HT_F32, HT_F16, HT_BF16 = 0, 1, 2
HT_OK = 0
HT_ERR_INVALID_ARG, HT_ERR_UNSUPPORTED, HT_ERR_BAD_TREE, HT_ERR_WORKSPACE, HT_ERR_CUDA, HT_ERR_TIMEOUT = range(1, 7)
HT_STATUS_OK, HT_STATUS_BAD_TREE, HT_STATUS_BAD_LEN, HT_STATUS_BAD_PATH, HT_STATUS_PATH_TOO_LONG = range(5)
HT_ATTN_FORCE_SIMT = 1
HT_ATTN_WORKSPACE_CLEAN = 2
HT_ATTN_CONTEXT_FINAL = 4
HT_ATTN_TEST_SHORT_WAITS = 0x80000000
HT_STATUS_BAD_PAGE, HT_STATUS_TIMEOUT = 5, 6

EXPORTS = ("ht_version", "ht_last_error_string", "ht_transfer", "ht_tree_attention_workspace",
           "ht_tree_attention", "ht_verify_greedy", "ht_kv_compact", "ht_draft_tree", "ht_rope_kv_append", "ht_tree_attention_static",
           "ht_tree_attention_paged", "ht_rope_kv_append_paged", "ht_kv_compact_paged", "ht_tree_attention_launches",
           "ht_verify_greedy_compact")
HT_STATIC_SCRATCH_BYTES = 16 << 20

_DTYPES = {torch.float32: HT_F32, torch.float16: HT_F16, torch.bfloat16: HT_BF16}


class AttnDesc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("N", ctypes.c_int32), ("Hq", ctypes.c_int32),
                ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32), ("cap", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("scale", ctypes.c_float),
                ("kv_stride_b", ctypes.c_int64), ("kv_stride_h", ctypes.c_int64),
                ("num_splits", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class PagedDesc(ctypes.Structure):
    _fields_ = [("page_size", ctypes.c_int32), ("max_pages", ctypes.c_int32), ("n_pages", ctypes.c_int32),
                ("page_stride", ctypes.c_int64), ("head_stride", ctypes.c_int64)]


class CacheDesc(ctypes.Structure):
    _fields_ = [("layers", ctypes.c_int32), ("B", ctypes.c_int32), ("Hkv", ctypes.c_int32),
                ("cap", ctypes.c_int32), ("D", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("N", ctypes.c_int32), ("stride_layer", ctypes.c_int64),
                ("stride_b", ctypes.c_int64), ("stride_h", ctypes.c_int64)]


class HtError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__("libht error %d: %s" % (code, message))
        self.code = code


_lib = None


def load() -> ctypes.CDLL:
    """Load ``libht.so`` (built in-tree by ``paper_2404_12022_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libht.so is missing at %s: build it with `python -m paper_2404_12022_b200.build`; "
                "there is no fallback path" % LIB_PATH)
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        lib.ht_version.restype = i32
        lib.ht_last_error_string.restype = ctypes.c_char_p
        lib.ht_transfer.restype = i32
        lib.ht_transfer.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp]
        lib.ht_tree_attention_workspace.restype = sz
        lib.ht_tree_attention_workspace.argtypes = [ctypes.POINTER(AttnDesc)]
        lib.ht_tree_attention_launches.restype = i32
        lib.ht_tree_attention_launches.argtypes = [ctypes.POINTER(AttnDesc)]
        lib.ht_tree_attention.restype = i32
        lib.ht_tree_attention.argtypes = [ctypes.POINTER(AttnDesc), vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        lib.ht_tree_attention_static.restype = i32
        lib.ht_tree_attention_static.argtypes = [ctypes.POINTER(AttnDesc), vp, vp, vp, vp, vp, vp, vp, vp]
        lib.ht_tree_attention_paged.restype = i32
        lib.ht_tree_attention_paged.argtypes = [ctypes.POINTER(AttnDesc), ctypes.POINTER(PagedDesc), vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        lib.ht_rope_kv_append_paged.restype = i32
        lib.ht_rope_kv_append_paged.argtypes = [ctypes.POINTER(AttnDesc), ctypes.POINTER(PagedDesc), vp, vp, vp, vp, vp, vp,
                                                ctypes.c_float, vp, vp, vp, vp, vp]
        lib.ht_kv_compact_paged.restype = i32
        lib.ht_kv_compact_paged.argtypes = [vp, vp, ctypes.POINTER(CacheDesc), ctypes.POINTER(PagedDesc), vp, vp, vp, vp, i32,
                                            vp, vp, vp]
        lib.ht_verify_greedy.restype = i32
        lib.ht_verify_greedy.argtypes = [vp, i32, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        lib.ht_verify_greedy_compact.restype = i32
        lib.ht_verify_greedy_compact.argtypes = [vp, i32, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp,
                                                 vp, vp, ctypes.POINTER(CacheDesc), vp, vp, vp, vp]
        lib.ht_kv_compact.restype = i32
        lib.ht_kv_compact.argtypes = [vp, vp, ctypes.POINTER(CacheDesc), vp, vp, vp, i32, vp, vp, vp]
        lib.ht_draft_tree.restype = i32
        lib.ht_draft_tree.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp]
        lib.ht_rope_kv_append.restype = i32
        lib.ht_rope_kv_append.argtypes = [ctypes.POINTER(AttnDesc), vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, vp]
        _lib = lib
    return _lib


def _check(rc: int):
    if rc != HT_OK:
        raise HtError(rc, load().ht_last_error_string().decode())


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _need(t: torch.Tensor, dtype=None, name="tensor"):
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor (this library has no CPU path)" % name)
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    if dtype is not None and t.dtype != dtype:
        raise ValueError("%s must be %s" % (name, dtype))


def transfer(h_src: torch.Tensor, W: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """h_src [B, d], W [k, d, d] -> out [B, k, d] (same dtype)."""
    _need(h_src, name="h_src")
    _need(W, h_src.dtype, "W")
    B, d = h_src.shape
    k = W.shape[0]
    if tuple(W.shape) != (k, d, d):
        raise ValueError("W must be [k, d, d]")
    if out is None:
        out = torch.empty((B, k, d), dtype=h_src.dtype, device=h_src.device)
    _need(out, h_src.dtype, "out")
    _check(load().ht_transfer(_ptr(h_src), _ptr(W), _ptr(out), B, k, d, _DTYPES[h_src.dtype], _stream()))
    return out


def make_attn_desc(q: torch.Tensor, k_cache: torch.Tensor, scale: float = 0.0, num_splits: int = 0,
                   flags: int = 0) -> AttnDesc:
    B, N, Hq, D = q.shape
    Bc, Hkv, cap, Dc = k_cache.shape
    if (Bc, Dc) != (B, D):
        raise ValueError("cache shape does not match q")
    if k_cache.stride(3) != 1 or k_cache.stride(2) != D:
        raise ValueError("cache rows must be contiguous and D apart")
    return AttnDesc(B, N, Hq, Hkv, D, cap, _DTYPES[q.dtype], float(scale), k_cache.stride(0),
                    k_cache.stride(1), num_splits, flags)


def tree_attention_launches(desc: AttnDesc) -> int:
    """Kernels of this library that one ``tree_attention`` call with this descriptor enqueues."""
    return int(load().ht_tree_attention_launches(ctypes.byref(desc)))


def tree_attention_workspace(desc: AttnDesc) -> int:
    return int(load().ht_tree_attention_workspace(ctypes.byref(desc)))


def tree_attention(q, k_cache, v_cache, kv_len, parent, out=None, workspace=None, status=None,
                   scale: float = 0.0, num_splits: int = 0, flags: int = 0):
    """q [B, N, Hq, D]; caches [B, Hkv, cap, D] (may be strided views over b / head);
    kv_len [B] int32; parent [B, N] int32.  Returns (out, status)."""
    _need(q, name="q")
    _need(kv_len, torch.int32, "kv_len")
    _need(parent, torch.int32, "parent")
    if not (k_cache.is_cuda and v_cache.is_cuda) or k_cache.dtype != q.dtype or v_cache.dtype != q.dtype:
        raise ValueError("caches must be CUDA tensors of q's dtype")
    if k_cache.stride() != v_cache.stride() or k_cache.shape != v_cache.shape:
        raise ValueError("k_cache and v_cache must share shape and strides")
    desc = make_attn_desc(q, k_cache, scale, num_splits, flags)
    B, N = desc.B, desc.N
    if tuple(parent.shape) != (B, N) or tuple(kv_len.shape) != (B,):
        raise ValueError("parent must be [B, N] and kv_len [B]")
    if out is None:
        out = torch.empty_like(q)
    _need(out, q.dtype, "out")
    if status is None:
        status = torch.empty(B, dtype=torch.int32, device=q.device)
    need = tree_attention_workspace(desc)
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().ht_tree_attention(ctypes.byref(desc), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(kv_len),
                                    _ptr(parent), _ptr(out), _ptr(workspace), ws_bytes, _ptr(status), _stream()))
    return out, status


def tree_attention_paged(q, k_pages, v_pages, block_table, kv_len, parent, out=None, workspace=None, status=None,
                         scale: float = 0.0, flags: int = 0):
    """q [B, N, Hq, D]; page pools [n_pages, Hkv, page_size, D] (may be strided over page / head);
    block_table [B, max_pages] int32; kv_len [B] int32; parent [B, N] int32.  Returns (out, status)."""
    _need(q, name="q")
    _need(block_table, torch.int32, "block_table")
    _need(kv_len, torch.int32, "kv_len")
    _need(parent, torch.int32, "parent")
    if not (k_pages.is_cuda and v_pages.is_cuda) or k_pages.dtype != q.dtype or v_pages.dtype != q.dtype:
        raise ValueError("page pools must be CUDA tensors of q's dtype")
    if k_pages.stride() != v_pages.stride() or k_pages.shape != v_pages.shape:
        raise ValueError("k_pages and v_pages must share shape and strides")
    B, N, Hq, D = q.shape
    n_pages, Hkv, page_size, Dp = k_pages.shape
    if Dp != D or k_pages.stride(3) != 1 or k_pages.stride(2) != D:
        raise ValueError("page rows must be contiguous and D apart")
    if block_table.dim() != 2 or block_table.shape[0] != B or tuple(parent.shape) != (B, N) or tuple(kv_len.shape) != (B,):
        raise ValueError("block_table must be [B, max_pages], parent [B, N], kv_len [B]")
    max_pages = block_table.shape[1]
    desc = AttnDesc(B, N, Hq, Hkv, D, max_pages * page_size, _DTYPES[q.dtype], scale, 0, 0, 0, flags)
    pages = PagedDesc(page_size, max_pages, n_pages, k_pages.stride(0), k_pages.stride(1))
    if out is None:
        out = torch.empty_like(q)
    _need(out, q.dtype, "out")
    if status is None:
        status = torch.empty(B, dtype=torch.int32, device=q.device)
    need = tree_attention_workspace(desc)
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().ht_tree_attention_paged(ctypes.byref(desc), ctypes.byref(pages), _ptr(q), _ptr(k_pages), _ptr(v_pages),
                                          _ptr(block_table), _ptr(kv_len), _ptr(parent), _ptr(out), _ptr(workspace),
                                          ws_bytes, _ptr(status), _stream()))
    return out, status


def tree_attention_static(q, k_cache, v_cache, kv_len, parent, out=None, status=None, scale: float = 0.0,
                          num_splits: int = 0):
    """Tree attention for callers that cannot allocate scratch: same results as
    ``tree_attention``, with the split partials in the library's built-in array (at most
    ``HT_STATIC_SCRATCH_BYTES``; larger problems raise).  Calls must not overlap on the GPU.
    ``out`` and ``status`` may be passed in so that the call itself allocates nothing."""
    _need(q, name="q")
    _need(kv_len, torch.int32, "kv_len")
    _need(parent, torch.int32, "parent")
    desc = make_attn_desc(q, k_cache, scale, num_splits, 0)
    if out is None:
        out = torch.empty_like(q)
    if status is None:
        status = torch.empty(desc.B, dtype=torch.int32, device=q.device)
    _check(load().ht_tree_attention_static(ctypes.byref(desc), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(kv_len),
                                           _ptr(parent), _ptr(out), _ptr(status), _stream()))
    return out, status


def verify_greedy(logits, tokens, parent, root_pred=None, max_path: int = 8, accept_len=None):
    """logits [B, N, V]; tokens [B, T] int32; parent [B, N] int32; root_pred [B] int32 or None.
    ``accept_len`` [B] int32, if given, must hold zeros or what an earlier call left in it (the kernel counts
    arrivals in its upper bits); by default a zeroed tensor is made.
    Returns (pred [B, N], accept_len [B], accept_path [B, max_path], next_token [B], status [B])."""
    _need(logits, name="logits")
    _need(tokens, torch.int32, "tokens")
    _need(parent, torch.int32, "parent")
    B, N, V = logits.shape
    T = tokens.shape[1]
    if tuple(parent.shape) != (B, N) or tokens.shape[0] != B:
        raise ValueError("parent must be [B, N] and tokens [B, T]")
    if root_pred is not None:
        _need(root_pred, torch.int32, "root_pred")
    dev = logits.device
    pred = torch.empty((B, N), dtype=torch.int32, device=dev)
    if accept_len is None:
        accept_len = torch.zeros(B, dtype=torch.int32, device=dev)
    else:
        _need(accept_len, torch.int32, "accept_len")
    accept_path = torch.empty((B, max_path), dtype=torch.int32, device=dev)
    next_token = torch.empty(B, dtype=torch.int32, device=dev)
    status = torch.empty(B, dtype=torch.int32, device=dev)
    _check(load().ht_verify_greedy(_ptr(logits), _DTYPES[logits.dtype], _ptr(tokens), _ptr(parent),
                                   _ptr(root_pred), B, N, T, V, max_path, _ptr(pred), _ptr(accept_len),
                                   _ptr(accept_path), _ptr(next_token), _ptr(status), _stream()))
    return pred, accept_len, accept_path, next_token, status


def verify_greedy_compact(logits, tokens, parent, root_pred, k_cache, v_cache, kv_len, max_path: int = 8, rows: int = 0,
                          accept_len=None):
    """Verification and compaction in one launch: ``verify_greedy`` followed by ``kv_compact`` on caches
    [layers, B, Hkv, cap, D].  ``rows``: logits rows per sequence whose argmax is taken (0 = the T tree rows).
    Returns (pred, accept_len, accept_path, next_token, status, new_kv_len, compact_status)."""
    _need(logits, name="logits")
    _need(tokens, torch.int32, "tokens")
    _need(parent, torch.int32, "parent")
    _need(kv_len, torch.int32, "kv_len")
    B, N, V = logits.shape
    T = tokens.shape[1]
    if tuple(parent.shape) != (B, N) or tokens.shape[0] != B:
        raise ValueError("parent must be [B, N] and tokens [B, T]")
    if root_pred is not None:
        _need(root_pred, torch.int32, "root_pred")
    if not (k_cache.is_cuda and v_cache.is_cuda) or k_cache.dtype != v_cache.dtype:
        raise ValueError("caches must be CUDA tensors of one dtype")
    if k_cache.stride() != v_cache.stride() or k_cache.shape != v_cache.shape:
        raise ValueError("k_cache and v_cache must share shape and strides")
    layers, Bc, Hkv, cap, D = k_cache.shape
    if k_cache.stride(4) != 1 or k_cache.stride(3) != D or Bc != B:
        raise ValueError("cache rows must be contiguous and D apart, and the caches must hold B sequences")
    desc = CacheDesc(layers, B, Hkv, cap, D, _DTYPES[k_cache.dtype], N, k_cache.stride(0), k_cache.stride(1), k_cache.stride(2))
    dev = logits.device
    pred = torch.full((B, N), -1, dtype=torch.int32, device=dev)
    if accept_len is None:
        accept_len = torch.zeros(B, dtype=torch.int32, device=dev)
    else:
        _need(accept_len, torch.int32, "accept_len")
    accept_path = torch.empty((B, max_path), dtype=torch.int32, device=dev)
    next_token = torch.empty(B, dtype=torch.int32, device=dev)
    status = torch.empty(B, dtype=torch.int32, device=dev)
    new_kv_len = torch.empty(B, dtype=torch.int32, device=dev)
    compact_status = torch.empty(B, dtype=torch.int32, device=dev)
    _check(load().ht_verify_greedy_compact(_ptr(logits), _DTYPES[logits.dtype], _ptr(tokens), _ptr(parent), _ptr(root_pred),
                                           B, N, T, V, max_path, rows, _ptr(pred), _ptr(accept_len), _ptr(accept_path),
                                           _ptr(next_token), _ptr(status), _ptr(k_cache), _ptr(v_cache), ctypes.byref(desc),
                                           _ptr(kv_len), _ptr(new_kv_len), _ptr(compact_status), _stream()))
    return pred, accept_len, accept_path, next_token, status, new_kv_len, compact_status


def kv_compact(k_cache, v_cache, n_rows: int, kv_len, accept_len, accept_path, new_kv_len=None,
               status=None):
    """In-place compaction of caches [layers, B, Hkv, cap, D].  Returns (new_kv_len, status)."""
    if not (k_cache.is_cuda and v_cache.is_cuda) or k_cache.dtype != v_cache.dtype:
        raise ValueError("caches must be CUDA tensors of one dtype")
    if k_cache.stride() != v_cache.stride() or k_cache.shape != v_cache.shape:
        raise ValueError("k_cache and v_cache must share shape and strides")
    layers, B, Hkv, cap, D = k_cache.shape
    if k_cache.stride(4) != 1 or k_cache.stride(3) != D:
        raise ValueError("cache rows must be contiguous and D apart")
    _need(kv_len, torch.int32, "kv_len")
    _need(accept_len, torch.int32, "accept_len")
    _need(accept_path, torch.int32, "accept_path")
    max_path = accept_path.shape[1]
    desc = CacheDesc(layers, B, Hkv, cap, D, _DTYPES[k_cache.dtype], int(n_rows), k_cache.stride(0),
                     k_cache.stride(1), k_cache.stride(2))
    dev = k_cache.device
    if new_kv_len is None:
        new_kv_len = torch.empty(B, dtype=torch.int32, device=dev)
    if status is None:
        status = torch.empty(B, dtype=torch.int32, device=dev)
    _check(load().ht_kv_compact(_ptr(k_cache), _ptr(v_cache), ctypes.byref(desc), _ptr(kv_len),
                                _ptr(accept_len), _ptr(accept_path), max_path, _ptr(new_kv_len),
                                _ptr(status), _stream()))
    return new_kv_len, status


def draft_tree(logits, first_row: int, P: int, K: int, tmpl_parent, tmpl_rank, root_token, base_pos):
    """logits [B, rows, V]; pseudo position i (1..P) is row first_row + i - 1; tmpl_parent, tmpl_rank
    [T] int32; root_token [B] int32 or None; base_pos [B] int32.
    Returns (topk [B, P, K], tokens [B, T], pos [B, T], status [B])."""
    _need(logits, name="logits")
    _need(tmpl_parent, torch.int32, "tmpl_parent")
    _need(tmpl_rank, torch.int32, "tmpl_rank")
    _need(base_pos, torch.int32, "base_pos")
    if root_token is not None:
        _need(root_token, torch.int32, "root_token")
    B, rows, V = logits.shape
    T = tmpl_parent.shape[0]
    dev = logits.device
    topk = torch.empty((B, P, K), dtype=torch.int32, device=dev)
    tokens = torch.empty((B, T), dtype=torch.int32, device=dev)
    pos = torch.empty((B, T), dtype=torch.int32, device=dev)
    status = torch.empty(B, dtype=torch.int32, device=dev)
    _check(load().ht_draft_tree(_ptr(logits), _DTYPES[logits.dtype], B, rows, V, first_row, P, K, _ptr(tmpl_parent),
                                _ptr(tmpl_rank), T, _ptr(root_token), _ptr(base_pos), _ptr(topk), _ptr(tokens),
                                _ptr(pos), _ptr(status), _stream()))
    return topk, tokens, pos, status


def rope_kv_append(q_in, k_in, v_in, pos, kv_len, k_cache, v_cache, rope_base: float = 10000.0, q_out=None):
    """q_in [B, N, Hq, D]; k_in, v_in [B, N, Hkv, D]; pos [B, N] int32; kv_len [B] int32; caches
    [B, Hkv, cap, D] (written in place at rows kv_len[b] + r).  Returns (q_out, status)."""
    _need(q_in, name="q_in")
    _need(k_in, q_in.dtype, "k_in")
    _need(v_in, q_in.dtype, "v_in")
    _need(pos, torch.int32, "pos")
    _need(kv_len, torch.int32, "kv_len")
    desc = make_attn_desc(q_in, k_cache)
    if q_out is None:
        q_out = torch.empty_like(q_in)
    status = torch.empty(desc.B, dtype=torch.int32, device=q_in.device)
    _check(load().ht_rope_kv_append(ctypes.byref(desc), _ptr(q_in), _ptr(k_in), _ptr(v_in), _ptr(pos), _ptr(kv_len),
                                    float(rope_base), _ptr(q_out), _ptr(k_cache), _ptr(v_cache), _ptr(status), _stream()))
    return q_out, status


def rope_kv_append_paged(q_in, k_in, v_in, pos, kv_len, block_table, k_pages, v_pages, rope_base: float = 10000.0,
                         q_out=None):
    """As ``rope_kv_append`` with the caches as page pools [n_pages, Hkv, page_size, D] (written in place at the
    logical rows kv_len[b] + r through block_table [B, max_pages]).  Returns (q_out, status)."""
    _need(q_in, name="q_in")
    _need(k_in, q_in.dtype, "k_in")
    _need(v_in, q_in.dtype, "v_in")
    _need(pos, torch.int32, "pos")
    _need(kv_len, torch.int32, "kv_len")
    _need(block_table, torch.int32, "block_table")
    B, N, Hq, D = q_in.shape
    n_pages, Hkv, page_size, Dp = k_pages.shape
    if Dp != D or k_pages.stride(3) != 1 or k_pages.stride(2) != D or k_pages.stride() != v_pages.stride():
        raise ValueError("page rows must be contiguous and D apart, K and V pools alike")
    max_pages = block_table.shape[1]
    desc = AttnDesc(B, N, Hq, Hkv, D, max_pages * page_size, _DTYPES[q_in.dtype], 0.0, 0, 0, 0, 0)
    pages = PagedDesc(page_size, max_pages, n_pages, k_pages.stride(0), k_pages.stride(1))
    if q_out is None:
        q_out = torch.empty_like(q_in)
    status = torch.empty(B, dtype=torch.int32, device=q_in.device)
    _check(load().ht_rope_kv_append_paged(ctypes.byref(desc), ctypes.byref(pages), _ptr(q_in), _ptr(k_in), _ptr(v_in),
                                          _ptr(pos), _ptr(kv_len), _ptr(block_table), float(rope_base), _ptr(q_out),
                                          _ptr(k_pages), _ptr(v_pages), _ptr(status), _stream()))
    return q_out, status


def kv_compact_paged(k_pages, v_pages, block_table, n_rows: int, kv_len, accept_len, accept_path, new_kv_len=None,
                     status=None):
    """In-place compaction of page pools [layers, n_pages, Hkv, page_size, D] that share block_table
    [B, max_pages].  Returns (new_kv_len, status)."""
    if not (k_pages.is_cuda and v_pages.is_cuda) or k_pages.dtype != v_pages.dtype:
        raise ValueError("pools must be CUDA tensors of one dtype")
    if k_pages.stride() != v_pages.stride() or k_pages.shape != v_pages.shape:
        raise ValueError("k_pages and v_pages must share shape and strides")
    layers, n_pages, Hkv, page_size, D = k_pages.shape
    if k_pages.stride(4) != 1 or k_pages.stride(3) != D:
        raise ValueError("page rows must be contiguous and D apart")
    _need(block_table, torch.int32, "block_table")
    _need(kv_len, torch.int32, "kv_len")
    _need(accept_len, torch.int32, "accept_len")
    _need(accept_path, torch.int32, "accept_path")
    B, max_pages = block_table.shape
    max_path = accept_path.shape[1]
    desc = CacheDesc(layers, B, Hkv, max_pages * page_size, D, _DTYPES[k_pages.dtype], int(n_rows), k_pages.stride(0), 0, 0)
    pages = PagedDesc(page_size, max_pages, n_pages, k_pages.stride(1), k_pages.stride(2))
    dev = k_pages.device
    if new_kv_len is None:
        new_kv_len = torch.empty(B, dtype=torch.int32, device=dev)
    if status is None:
        status = torch.empty(B, dtype=torch.int32, device=dev)
    _check(load().ht_kv_compact_paged(_ptr(k_pages), _ptr(v_pages), ctypes.byref(desc), ctypes.byref(pages),
                                      _ptr(block_table), _ptr(kv_len), _ptr(accept_len), _ptr(accept_path), max_path,
                                      _ptr(new_kv_len), _ptr(status), _stream()))
    return new_kv_len, status
