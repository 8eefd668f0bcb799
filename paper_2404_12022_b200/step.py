"""One tree-verify step as a fixed sequence of library calls.

``VerifyStep`` owns the descriptors, outputs and workspace of a workload so that a step is
nothing but C-ABI calls on the current stream: per layer ``ht_tree_attention`` (with the
pseudo rows joining after the transfer layer), one ``ht_transfer``, one ``ht_verify_greedy``
and one ``ht_kv_compact`` over all layers (``fused=True``: the last two as one launch,
``ht_verify_greedy_compact``).  The dense parts of the
transformer layer between those calls are outside this library; their outputs (q, the new
K/V rows, the logits) are inputs here.
"""
from __future__ import annotations

import ctypes
from typing import List, Optional

import torch

from . import binding as hb
from .workloads import Inputs


class VerifyStep:
    def __init__(self, inp: Inputs, num_splits: int = 0, flags: int = 0, fused: bool = False):
        # Verification and compaction as one launch (ht_verify_greedy_compact) or as two calls.  The chain of
        # dependent steps is the same either way (argmax, count, path search, rows), and so is the time within a
        # microsecond or two: replayed in the graph of a whole step the two calls come out ahead (config 2: 51.5
        # against 55.7 us per step; config 3's 32 layers: 19.9 against 21.5 us for the pair), so they are the default.
        self.fused = fused
        w = inp.w
        self.inp = inp
        self.w = w
        self.lib = hb.load()
        dev = inp.k_cache.device
        self.layers = inp.k_cache.shape[0]
        self.descs: List[hb.AttnDesc] = []
        self.parents: List[torch.Tensor] = []
        self.outs: List[torch.Tensor] = []
        ws_bytes = 0
        for i in range(self.layers):
            q = inp.q[i]
            # the step owns its workspace: zeroed below, and left clean by every call; lengths, trees and context
            # rows are final long before a layer's call (the compaction moves rows at or behind the lengths only)
            desc = hb.make_attn_desc(q, inp.k_cache[i], 0.0, num_splits,
                                     flags | hb.HT_ATTN_WORKSPACE_CLEAN | hb.HT_ATTN_CONTEXT_FINAL)
            self.descs.append(desc)
            self.parents.append(inp.parent if q.shape[1] == w.N else inp.parent_tree)
            self.outs.append(torch.empty_like(q))
            ws_bytes = max(ws_bytes, hb.tree_attention_workspace(desc))
        self.workspace = torch.zeros(max(ws_bytes, 16), dtype=torch.uint8, device=dev)
        self.ws_bytes = ws_bytes
        self.attn_status = torch.zeros((self.layers, w.B), dtype=torch.int32, device=dev)
        self.pseudo = torch.empty((w.B, w.k, w.d), dtype=inp.h_src.dtype, device=dev)
        self.pred = torch.empty((w.B, w.N), dtype=torch.int32, device=dev)
        self.accept_len = torch.zeros(w.B, dtype=torch.int32, device=dev)     # zero once: the kernel leaves a length in it each time
        self.accept_path = torch.empty((w.B, w.max_path), dtype=torch.int32, device=dev)
        self.next_token = torch.empty(w.B, dtype=torch.int32, device=dev)
        self.verify_status = torch.empty(w.B, dtype=torch.int32, device=dev)
        self.new_kv_len = torch.empty(w.B, dtype=torch.int32, device=dev)
        self.compact_status = torch.empty(w.B, dtype=torch.int32, device=dev)
        kc = inp.k_cache
        self.cache_desc = hb.CacheDesc(kc.shape[0], w.B, w.Hkv, kc.shape[3], w.D, hb._DTYPES[kc.dtype], w.N,
                                       kc.stride(0), kc.stride(1), kc.stride(2))
        self.dtype_code = hb._DTYPES[kc.dtype]
        self.transfer_at = min(w.transfer_after_layer, self.layers)
        self.launches_per_step = 0
        self.graph = None

    def attention(self, i: int, stream: int) -> None:
        inp = self.inp
        hb._check(self.lib.ht_tree_attention(
            ctypes.byref(self.descs[i]), inp.q[i].data_ptr(), inp.k_cache[i].data_ptr(),
            inp.v_cache[i].data_ptr(), inp.kv_len.data_ptr(), self.parents[i].data_ptr(),
            self.outs[i].data_ptr(), self.workspace.data_ptr(), self.ws_bytes,
            self.attn_status[i].data_ptr(), stream))

    def transfer(self, stream: int) -> None:
        inp, w = self.inp, self.w
        hb._check(self.lib.ht_transfer(inp.h_src.data_ptr(), inp.W.data_ptr(), self.pseudo.data_ptr(),
                                       w.B, w.k, w.d, self.dtype_code, stream))

    def verify(self, stream: int) -> None:
        inp, w = self.inp, self.w
        hb._check(self.lib.ht_verify_greedy(
            inp.logits.data_ptr(), hb._DTYPES[inp.logits.dtype], inp.tokens.data_ptr(), inp.parent.data_ptr(),
            None if inp.root_pred is None else inp.root_pred.data_ptr(), w.B, w.N, w.T, w.V, w.max_path,
            self.pred.data_ptr(), self.accept_len.data_ptr(), self.accept_path.data_ptr(),
            self.next_token.data_ptr(), self.verify_status.data_ptr(), stream))

    def compact(self, stream: int) -> None:
        inp = self.inp
        hb._check(self.lib.ht_kv_compact(
            inp.k_cache.data_ptr(), inp.v_cache.data_ptr(), ctypes.byref(self.cache_desc),
            inp.kv_len.data_ptr(), self.accept_len.data_ptr(), self.accept_path.data_ptr(), self.w.max_path,
            self.new_kv_len.data_ptr(), self.compact_status.data_ptr(), stream))

    def verify_compact(self, stream: int) -> None:
        """Verification (argmax of the tree rows only) and compaction as one launch."""
        inp, w = self.inp, self.w
        hb._check(self.lib.ht_verify_greedy_compact(
            inp.logits.data_ptr(), hb._DTYPES[inp.logits.dtype], inp.tokens.data_ptr(), inp.parent.data_ptr(),
            None if inp.root_pred is None else inp.root_pred.data_ptr(), w.B, w.N, w.T, w.V, w.max_path, 0,
            self.pred.data_ptr(), self.accept_len.data_ptr(), self.accept_path.data_ptr(),
            self.next_token.data_ptr(), self.verify_status.data_ptr(), inp.k_cache.data_ptr(), inp.v_cache.data_ptr(),
            ctypes.byref(self.cache_desc), inp.kv_len.data_ptr(), self.new_kv_len.data_ptr(),
            self.compact_status.data_ptr(), stream))

    def run(self, stream: Optional[int] = None, attn_hook=None) -> None:
        """Enqueue one whole step.  ``attn_hook(i, when)`` is called around each attention call
        (when = 0 before, 1 after) so that a caller can record events."""
        s = torch.cuda.current_stream().cuda_stream if stream is None else stream
        for i in range(self.layers):
            if i == self.transfer_at:
                self.transfer(s)
            if attn_hook:
                attn_hook(i, 0)
            self.attention(i, s)
            if attn_hook:
                attn_hook(i, 1)
        if self.transfer_at >= self.layers:
            self.transfer(s)
        if self.fused:
            self.verify_compact(s)
        else:
            self.verify(s)
            self.compact(s)

    def capture(self) -> None:
        """Record one whole step into a CUDA graph (after at least one eager ``run``, which does the
        library's once-per-device set-up).  ``replay`` then enqueues the step with a single launch:
        the same kernels on the same buffers, without per-call host work between them."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side), torch.cuda.graph(self.graph, stream=side):
            self.run(side.cuda_stream)
        torch.cuda.current_stream().wait_stream(side)

    def replay(self) -> None:
        self.graph.replay()

    # ---- algorithmic bytes (what each kernel must move at least once) ----
    def attention_bytes(self, i: int) -> int:
        w = self.w
        e = w.elem_bytes()
        rows = self.inp.q[i].shape[1]
        kv = sum(2 * w.Hkv * (L + rows) * w.D * e for L in w.kv_len)
        qo = 2 * w.B * rows * w.Hq * w.D * e
        return kv + qo + 4 * w.B * rows

    def attention_flops(self, i: int) -> int:
        w = self.w
        rows = self.inp.q[i].shape[1]
        return sum(4 * rows * w.Hq * (L + rows) * w.D for L in w.kv_len)

    def transfer_bytes(self) -> int:
        w = self.w
        e = w.elem_bytes()
        return w.k * w.d * w.d * e + w.B * w.d * e + w.B * w.k * w.d * e

    def verify_bytes(self) -> int:
        w = self.w
        return w.B * (w.T if self.fused else w.N) * w.V * w.elem_bytes()       # fused: the tree rows only

    def compact_bytes(self) -> int:
        w = self.w
        a = sum(self.inp.want_len)
        return 2 * 2 * self.layers * a * w.Hkv * w.D * w.elem_bytes()

    def step_bytes(self) -> int:
        return (sum(self.attention_bytes(i) for i in range(self.layers)) + self.transfer_bytes() +
                self.verify_bytes() + self.compact_bytes())
