"""ctypes front end of the CPU oracle (``ht_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's
CPU-baseline leg, never by the product package.  It compiles ``ht_oracle.c`` with gcc
on first use and marshals numpy arrays; every piece of arithmetic lives in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ht_oracle.c")
_LIB = os.path.join(_HERE, "libht_oracle.so")
_lock = threading.Lock()
_lib = None

OK, BAD_TREE, BAD_LEN, BAD_PATH, PATH_TOO_LONG, NOMEM = range(6)


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object beside its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-Wall", "-Wextra",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            _lib = ctypes.CDLL(build())
            _lib.ht_oracle_num_threads.restype = ctypes.c_int
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(_load().ht_oracle_num_threads())


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__("oracle returned error %d" % code)
        self.code = code


def _check(code):
    if code != OK:
        raise OracleError(code)


def transfer(h, W):
    """h [B, d], W [k, d, d] -> float64 [B, k, d]."""
    h = _f32(h)
    W = _f32(W)
    B, d = h.shape
    k = W.shape[0]
    assert W.shape == (k, d, d)
    out = np.empty((B, k, d), dtype=np.float64)
    _check(_load().ht_oracle_transfer(_p(h), _p(W), _p(out), B, k, d))
    return out


def _attn_args(q, k_cache, v_cache, kv_len, parent, scale):
    q = _f32(q)
    k_cache = _f32(k_cache)
    v_cache = _f32(v_cache)
    kv_len = _i32(kv_len)
    parent = _i32(parent)
    B, N, Hq, D = q.shape
    Bc, Hkv, cap, Dc = k_cache.shape
    assert (Bc, Dc) == (B, D) and v_cache.shape == k_cache.shape
    assert kv_len.shape == (B,) and parent.shape == (B, N)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    return q, k_cache, v_cache, kv_len, parent, B, N, Hq, Hkv, D, cap, float(scale)


def tree_attention(q, k_cache, v_cache, kv_len, parent, scale=None, sel=None):
    """Path-form tree attention.

    With ``sel`` None returns float64 [B, N, Hq, D]; otherwise ``sel`` is an int array
    [n, 3] of (b, h, r) triples and the result is [n, D].
    """
    q, k_cache, v_cache, kv_len, parent, B, N, Hq, Hkv, D, cap, scale = _attn_args(
        q, k_cache, v_cache, kv_len, parent, scale)
    lib = _load()
    if sel is None:
        out = np.empty((B, N, Hq, D), dtype=np.float64)
        sel_p, n_sel = None, 0
    else:
        sel = _i32(sel).reshape(-1, 3)
        assert sel.size == 0 or (sel.min() >= 0 and (sel.max(axis=0) < [B, Hq, N]).all())
        out = np.empty((sel.shape[0], D), dtype=np.float64)
        sel_p, n_sel = _p(sel), sel.shape[0]
    _check(lib.ht_oracle_tree_attention_rows(
        _p(q), _p(k_cache), _p(v_cache), _p(kv_len), _p(parent),
        B, N, Hq, Hkv, D, cap, ctypes.c_double(scale), sel_p, ctypes.c_long(n_sel), _p(out)))
    return out


def tree_attention_mask_form(q, k_cache, v_cache, kv_len, parent, scale=None):
    """Dense-mask form of the same definition; float64 [B, N, Hq, D]."""
    q, k_cache, v_cache, kv_len, parent, B, N, Hq, Hkv, D, cap, scale = _attn_args(
        q, k_cache, v_cache, kv_len, parent, scale)
    out = np.empty((B, N, Hq, D), dtype=np.float64)
    _check(_load().ht_oracle_tree_attention_mask(
        _p(q), _p(k_cache), _p(v_cache), _p(kv_len), _p(parent),
        B, N, Hq, Hkv, D, cap, ctypes.c_double(scale), _p(out)))
    return out


def row_argmax(logits):
    """logits [..., V] -> int32 [...]; lowest index on ties, NaN never wins."""
    logits = _f32(logits)
    V = logits.shape[-1]
    rows = int(np.prod(logits.shape[:-1], dtype=np.int64))
    pred = np.empty(logits.shape[:-1], dtype=np.int32)
    _check(_load().ht_oracle_row_argmax(_p(logits), ctypes.c_long(rows), V, _p(pred)))
    return pred


def _accept(fn, tokens, parent, pred, root_pred, max_path):
    tokens = _i32(tokens)
    parent = _i32(parent)
    pred = _i32(pred)
    B, T = tokens.shape
    N = parent.shape[1]
    assert parent.shape == (B, N) and pred.shape == (B, N) and T <= N
    rp = None if root_pred is None else _i32(root_pred)
    accept_len = np.empty(B, dtype=np.int32)
    accept_path = np.empty((B, max_path), dtype=np.int32)
    next_token = np.empty(B, dtype=np.int32)
    status = np.empty(B, dtype=np.int32)
    _check(fn(_p(tokens), _p(parent), _p(pred), None if rp is None else _p(rp),
              B, N, T, max_path, _p(accept_len), _p(accept_path), _p(next_token), _p(status)))
    return accept_len, accept_path, next_token, status


def accept_enumerate(tokens, parent, pred, root_pred, max_path):
    """Definition form of greedy acceptance (all root paths enumerated)."""
    return _accept(_load().ht_oracle_accept_enumerate, tokens, parent, pred, root_pred, max_path)


def accept_scan(tokens, parent, pred, root_pred, max_path):
    """Scan form of greedy acceptance."""
    return _accept(_load().ht_oracle_accept_scan, tokens, parent, pred, root_pred, max_path)


def verify_greedy(logits, tokens, parent, root_pred, max_path):
    """Row argmax followed by acceptance; returns pred, accept_len, accept_path, next_token, status."""
    pred = row_argmax(logits)
    a, p, n, s = accept_enumerate(tokens, parent, pred, root_pred, max_path)
    return pred, a, p, n, s


def kv_compact(k_cache, v_cache, n_rows, kv_len, accept_len, accept_path):
    """Compaction on copies of byte-viewable caches [layers, B, Hkv, cap, D].

    ``k_cache`` / ``v_cache`` are numpy arrays of any fixed-size element type (uint16 views
    of fp16 / bf16 storage included).  ``n_rows`` is N, the number of tree rows that sit
    behind each sequence's context.  Returns (k_new, v_new, new_kv_len, status).
    """
    k_new = np.array(k_cache, copy=True, order="C")
    v_new = np.array(v_cache, copy=True, order="C")
    layers, B, Hkv, cap, D = k_new.shape
    assert v_new.shape == k_new.shape and v_new.dtype == k_new.dtype
    kv_len = _i32(kv_len)
    accept_len = _i32(accept_len)
    accept_path = _i32(accept_path)
    max_path = accept_path.shape[1]
    new_len = np.empty(B, dtype=np.int32)
    status = np.empty(B, dtype=np.int32)
    _check(_load().ht_oracle_kv_compact(
        _p(k_new), _p(v_new), layers, B, Hkv, cap, D, k_new.dtype.itemsize, int(n_rows),
        _p(kv_len), _p(accept_len), _p(accept_path), max_path, _p(new_len), _p(status)))
    return k_new, v_new, new_len, status
