"""Seeded synthetic inputs for the tree-verify step (shapes of LLaMA-class decoding).

This module serves both the CUDA library's tests / benchmark and the CPU oracle's, and
therefore contains none of the method's arithmetic: no attention, no projection, no
argmax, no path search.  It only draws numbers, builds parent-index arrays and writes
planted values into logits.

Random numbers come from a counter-based generator: element ``i`` of stream ``s`` under
seed ``z`` is ``table[mix(z, s, i) >> 16]`` where ``table`` holds 65536 quantiles of the
standard normal and ``mix`` is two rounds of a 32-bit integer finaliser.  The value of an
element depends only on (seed, stream, index), so any slice can be regenerated on the
host and is bit-identical to the same slice generated on the GPU (integer ops and a
table lookup only; the table is computed once on the CPU and copied).

Where the paper evaluates on XSum / Gsm8k prompts with LLaMA-2-Chat / Vicuna weights,
these inputs stand in: only tensor shapes, tree shapes and value distributions follow
those workloads.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence

import numpy as np
import torch

_MASK32 = 0xFFFFFFFF
_TABLE_BITS = 16
_table_cpu: Optional[torch.Tensor] = None
_table_dev = {}


def _normal_table(device) -> torch.Tensor:
    """65536 standard-normal quantiles (mid-points), float32, cached per device."""
    global _table_cpu
    if _table_cpu is None:
        n = 1 << _TABLE_BITS
        u = (torch.arange(n, dtype=torch.float64) + 0.5) / n
        _table_cpu = torch.special.ndtri(u).to(torch.float32)
    key = str(device)
    if key not in _table_dev:
        _table_dev[key] = _table_cpu.to(device)
    return _table_dev[key]


def _mul32(x: torch.Tensor, c: int) -> torch.Tensor:
    """(x * c) mod 2^32 for int64 tensors holding values below 2^32, without overflow."""
    lo = (x & 0xFFFF) * c
    hi = (((x >> 16) * c) & 0xFFFF) << 16
    return (lo + hi) & _MASK32


def _mix32(x: torch.Tensor) -> torch.Tensor:
    x = x ^ (x >> 16)
    x = _mul32(x, 0x85EBCA6B)
    x = x ^ (x >> 13)
    x = _mul32(x, 0xC2B2AE35)
    x = x ^ (x >> 16)
    return x


def hashed_normal(seed: int, stream: int, start: int, count: int, device="cpu",
                  std: float = 1.0, dtype=torch.float32, chunk: int = 1 << 25) -> torch.Tensor:
    """``count`` draws of N(0, std^2), elements [start, start+count) of a stream, as ``dtype``."""
    table = _normal_table(device)
    out = torch.empty(count, dtype=dtype, device=device)
    salt = ((seed * 0x9E3779B1) ^ (stream * 0x7F4A7C15) ^ 0x5BD1E995) & _MASK32
    for off in range(0, count, chunk):
        n = min(chunk, count - off)
        idx = torch.arange(start + off, start + off + n, dtype=torch.int64, device=device)
        key = _mix32((idx & _MASK32) ^ salt)
        key = _mix32(key ^ ((idx >> 32) & _MASK32) ^ ((stream * 0x632BE5AB) & _MASK32))
        vals = table[key >> (32 - _TABLE_BITS)]
        if std != 1.0:
            vals = vals * std
        out[off:off + n] = vals.to(dtype)
    return out


def normal_tensor(seed: int, stream: int, shape: Sequence[int], device="cpu", std: float = 1.0,
                  dtype=torch.float32) -> torch.Tensor:
    count = int(np.prod(shape, dtype=np.int64))
    return hashed_normal(seed, stream, 0, count, device, std, dtype).reshape(*shape)


# --------------------------------------------------------------------------------------
# Trees as parent-index arrays (ancestor-first order; -1 attaches a node to the context)
# --------------------------------------------------------------------------------------

def full_binary_tree(depth: int) -> np.ndarray:
    """Root plus ``depth`` levels of branching 2 in BFS order (15 nodes for depth 3)."""
    n = (1 << (depth + 1)) - 1
    parent = np.array([(i - 1) // 2 for i in range(n)], dtype=np.int32)
    parent[0] = -1
    return parent


def level_tree(level_sizes: Sequence[int], rng: Optional[np.random.Generator] = None,
               root: bool = False) -> np.ndarray:
    """BFS tree with given level sizes.

    With ``rng`` None, level ``i+1`` is split evenly among the nodes of level ``i`` (sizes must
    divide); otherwise each node draws its parent uniformly from the previous level.  The
    first level attaches to the context (parent -1) unless ``root`` puts a single root node
    above it.
    """
    parent: List[int] = []
    prev: List[int] = []
    if root:
        parent.append(-1)
        prev = [0]
    for size in level_sizes:
        first = len(parent)
        for j in range(size):
            if not prev:
                parent.append(-1)
            elif rng is None:
                parent.append(prev[j * len(prev) // size])
            else:
                parent.append(int(prev[int(rng.integers(len(prev)))]))
        prev = list(range(first, first + size))
    return np.array(parent, dtype=np.int32)


def truncated_cartesian_tree(widths: Sequence[int], total: int) -> np.ndarray:
    """Root, then levels of ``widths[i]`` children per node in BFS order, cut to ``total`` nodes."""
    sizes, n = [], 1
    for w in widths:
        n *= w
        sizes.append(n)
    return level_tree(sizes, None, root=True)[:total]


def random_depth_tree(n_nodes: int, max_depth: int, rng: np.random.Generator) -> np.ndarray:
    """Node 0 is the root; every later node's parent is uniform among earlier nodes whose depth
    (root = 0) is below ``max_depth``."""
    parent = np.full(n_nodes, -1, dtype=np.int32)
    depth = np.zeros(n_nodes, dtype=np.int32)
    for i in range(1, n_nodes):
        cand = np.nonzero(depth[:i] < max_depth)[0]
        p = int(cand[int(rng.integers(len(cand)))])
        parent[i] = p
        depth[i] = depth[p] + 1
    return parent


def append_pseudo_rows(parent_tree: np.ndarray, src: int, n_pseudo: int) -> np.ndarray:
    """Pseudo positions as ordinary rows behind the tree: the first hangs off ``src`` (the
    node whose hidden state is transferred), each later one off its predecessor."""
    T = len(parent_tree)
    extra = [src] + [T + i for i in range(n_pseudo - 1)]
    return np.concatenate([parent_tree, np.array(extra[:n_pseudo], dtype=np.int32)]).astype(np.int32)


def append_pseudo_rows_per_node(parent_tree: np.ndarray, k: int) -> np.ndarray:
    """Pseudo positions for EVERY tree node (each token of the input gets its pseudo states): behind
    the T tree rows, node c owns rows T + c k ... T + c k + k - 1; the first hangs off c, each later
    one off its predecessor.  T (1 + k) rows in all."""
    T = len(parent_tree)
    extra = []
    for c in range(T):
        for i in range(k):
            extra.append(c if i == 0 else T + c * k + i - 1)
    return np.concatenate([parent_tree, np.array(extra, dtype=np.int32)]).astype(np.int32)


def node_depths(parent: np.ndarray) -> np.ndarray:
    depth = np.zeros(len(parent), dtype=np.int32)
    for i, p in enumerate(parent):
        depth[i] = 1 if p < 0 else depth[p] + 1
    return depth


# --------------------------------------------------------------------------------------
# Draft tokens and planted logits
# --------------------------------------------------------------------------------------

PLANTED_LOGIT = 8.0  # above every quantile in the table (|x| < 4.4), exact in fp16 / bf16


def draft_tokens(parent_tree: np.ndarray, V: int, rng: np.random.Generator) -> np.ndarray:
    """One token per tree node; siblings (top-level nodes included) get distinct tokens."""
    T = len(parent_tree)
    tokens = np.zeros(T, dtype=np.int32)
    groups = {}
    for c, p in enumerate(parent_tree):
        groups.setdefault(int(p), []).append(c)
    for members in groups.values():
        picks = rng.choice(V, size=len(members), replace=False)
        for c, t in zip(members, picks):
            tokens[c] = int(t)
    return tokens


def plant_acceptance(logits_b: torch.Tensor, tokens: np.ndarray, parent_tree: np.ndarray,
                     want_len: int, use_root_pred: bool, V: int,
                     rng: np.random.Generator):
    """Write large logits so that exactly one root path of ``want_len`` nodes carries the
    tokens a greedy decoder would emit, and nothing longer does.

    Returns (root_pred or None, planted path as a list).  ``logits_b`` is [N, V] and is
    modified in place.  Only stores are performed here; nobody's argmax is evaluated.
    """
    T = len(parent_tree)
    depth = node_depths(parent_tree)
    children = {}
    for c, p in enumerate(parent_tree):
        children.setdefault(int(p), []).append(c)
    if not use_root_pred:
        want_len = max(want_len, 1)
    want_len = min(want_len, int(depth.max()))
    path: List[int] = []
    if want_len > 0:
        ends = np.nonzero(depth == want_len)[0]
        c = int(ends[int(rng.integers(len(ends)))])
        while c >= 0:
            path.append(c)
            c = int(parent_tree[c])
        path.reverse()

    def other_token(avoid):
        avoid = set(int(a) for a in avoid)
        while True:
            t = int(rng.integers(V))
            if t not in avoid:
                return t

    root_pred = None
    top_tokens = [tokens[c] for c in children.get(-1, [])]
    if use_root_pred:
        root_pred = int(tokens[path[0]]) if path else other_token(top_tokens)
    for a, nxt in zip(path[:-1], path[1:]):
        logits_b[a, int(tokens[nxt])] = PLANTED_LOGIT
    if path:
        last = path[-1]
        kids = [tokens[c] for c in children.get(last, []) if c < T]
        logits_b[last, other_token(kids)] = PLANTED_LOGIT
    return root_pred, path


# --------------------------------------------------------------------------------------
# Workload descriptions
# --------------------------------------------------------------------------------------

@dataclasses.dataclass
class Workload:
    name: str
    layers: int
    B: int
    Hq: int
    Hkv: int
    D: int
    dtype: str                      # "f32" | "f16" | "bf16"
    kv_len: List[int]               # context length per sequence
    tree: str                       # "binary3" | "forest4322" | "forest4322_random" | "cart842_64" | "random_depth6"
    T: int
    P: int
    d: int
    k: int
    V: int
    w_std: float
    transfer_after_layer: int       # pseudo rows take part in attention from the next layer on
    use_root_pred: bool
    want_len: Optional[List[int]]   # seeded accepted length per sequence (None: drawn 0..4)
    seed: int
    max_path: int = 8
    per_node: bool = False          # pseudo rows hang off every tree node (P = T k) instead of one source node

    @property
    def N(self) -> int:
        return self.T + self.P

    @property
    def cap(self) -> int:
        need = max(self.kv_len) + self.N
        return (need + 127) // 128 * 128

    def rows_at_layer(self, layer: int) -> int:
        """Query rows taking part in attention at 0-based ``layer``."""
        return self.N if layer >= self.transfer_after_layer else self.T

    def torch_dtype(self):
        return {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}[self.dtype]

    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2


def _seed(cfg_index: int, point: int = 0) -> int:
    return 12022 * 100 + cfg_index + 1000 * point


def config_c1(want_len: int = 2) -> Workload:
    return Workload("c1_tiny_fp32", 1, 1, 4, 4, 64, "f32", [128], "binary3", 15, 3,
                    256, 3, 1000, 1.0 / 16.0, 0, False, [want_len], _seed(1, want_len))


def config_c2() -> Workload:
    return Workload("c2_llama7b_layer_fp16", 1, 1, 32, 32, 128, "f16", [1024], "forest4322", 88, 3,
                    4096, 3, 32000, 0.02, 0, True, None, _seed(2))


def config_c3(layers: int = 32, kv: int = 4096, B: int = 4) -> Workload:
    return Workload("c3_llama7b_step_bf16", layers, B, 32, 32, 128, "bf16", [kv] * B,
                    "forest4322_random", 88, 3, 4096, 3, 32000, 0.02, layers // 2, True, None,
                    _seed(3))


def config_c4(B: int = 8, lo: int = 512, hi: int = 8192) -> Workload:
    rng = np.random.Generator(np.random.Philox(_seed(4)))
    lens = [int(x) for x in rng.integers(lo, hi + 1, size=B)]
    return Workload("c4_llama13b_ragged_bf16", 1, B, 40, 40, 128, "bf16", lens, "cart842_64", 64, 4,
                    5120, 4, 32000, 0.02, 0, True, None, _seed(4))


def per_node_variant(w: Workload) -> Workload:
    """The same configuration with pseudo states for every tree node: P = T k pseudo rows, N = T (1 + k)
    query rows, and B T source rows for the projection."""
    return dataclasses.replace(w, name=w.name + "_per_node", P=w.T * w.k, per_node=True)


def config_c5(kv: int, T: int, B: int) -> Workload:
    point = [512, 2048, 8192, 32768].index(kv) * 16 + [16, 64, 128, 256].index(T) * 4 + [1, 4, 16].index(B)
    return Workload("c5_gqa70b_kv%d_t%d_b%d" % (kv, T, B), 1, B, 64, 8, 128, "bf16", [kv] * B,
                    "random_depth6", T, 3, 8192, 3, 32000, 0.02, 0, True, None, _seed(5, point))


def c5_points():
    return [(kv, T, B) for kv in (512, 2048, 8192, 32768) for T in (16, 64, 128, 256)
            for B in (1, 4, 16)]


def build_tree(w: Workload, b: int, rng: np.random.Generator) -> np.ndarray:
    if w.tree == "binary3":
        return full_binary_tree(3)
    if w.tree == "forest4322":
        return level_tree([4, 12, 24, 48])
    if w.tree == "forest4322_random":
        return level_tree([4, 12, 24, 48], None if b == 0 else rng)
    if w.tree == "cart842_64":
        return truncated_cartesian_tree([8, 4, 2], 64)
    if w.tree == "random_depth6":
        return random_depth_tree(w.T, 6, rng)
    raise ValueError(w.tree)


@dataclasses.dataclass
class Inputs:
    w: Workload
    q: List[torch.Tensor]            # per layer [B, rows_at_layer, Hq, D]
    k_cache: torch.Tensor            # [layers, B, Hkv, cap, D]
    v_cache: torch.Tensor
    kv_len: torch.Tensor             # [B] int32
    parent: torch.Tensor             # [B, N] int32
    parent_tree: torch.Tensor        # [B, T] int32 (contiguous copy of the first T columns)
    tokens: torch.Tensor             # [B, T] int32
    logits: Optional[torch.Tensor]   # [B, N, V]
    root_pred: Optional[torch.Tensor]
    h_src: torch.Tensor              # [B, d] ([B T, d] with pseudo rows per node)
    W: Optional[torch.Tensor]        # [k, d, d]
    want_len: List[int]
    planted_path: List[List[int]]
    src_node: List[int]


def make_structure(w: Workload):
    """Host-side integer structure of a workload: trees, tokens, accepted lengths."""
    rng = np.random.Generator(np.random.Philox(w.seed))
    parents, trees, tokens, want, src = [], [], [], [], []
    for b in range(w.B):
        tree = build_tree(w, b, rng)
        assert len(tree) == w.T
        s = 0 if w.tree in ("binary3", "forest4322") else int(rng.integers(w.T))
        trees.append(tree)
        parents.append(append_pseudo_rows_per_node(tree, w.k) if w.per_node else append_pseudo_rows(tree, s, w.P))
        tokens.append(draft_tokens(tree, w.V, rng))
        src.append(s)
        want.append(int(w.want_len[b]) if w.want_len is not None else int(rng.integers(0, 5)))
    return rng, np.stack(parents), np.stack(trees), np.stack(tokens), want, src


def make_inputs(w: Workload, device="cpu", with_logits: bool = True, with_transfer: bool = True,
                layers: Optional[Sequence[int]] = None) -> Inputs:
    """Materialise a workload on ``device``.  ``layers`` restricts q / caches to the listed
    layer indices (values are those the full workload would hold for them)."""
    dt = w.torch_dtype()
    layer_ids = list(range(w.layers)) if layers is None else list(layers)
    rng, parent, trees, tokens, want, src = make_structure(w)
    cap, N = w.cap, w.N
    per_layer = w.B * w.Hkv * cap * w.D
    k_cache = torch.empty((len(layer_ids), w.B, w.Hkv, cap, w.D), dtype=dt, device=device)
    v_cache = torch.empty_like(k_cache)
    q = []
    for i, layer in enumerate(layer_ids):
        k_cache[i] = hashed_normal(w.seed, 1, layer * per_layer, per_layer, device, 1.0, dt).reshape(
            w.B, w.Hkv, cap, w.D)
        v_cache[i] = hashed_normal(w.seed, 2, layer * per_layer, per_layer, device, 1.0, dt).reshape(
            w.B, w.Hkv, cap, w.D)
        rows = w.rows_at_layer(layer)
        q_full = hashed_normal(w.seed, 3, layer * w.B * N * w.Hq * w.D, w.B * N * w.Hq * w.D, device,
                               1.0, dt).reshape(w.B, N, w.Hq, w.D)
        q.append(q_full[:, :rows].contiguous())
    logits = None
    root_pred = None
    planted = [[] for _ in range(w.B)]
    if with_logits:
        logits = normal_tensor(w.seed, 4, (w.B, N, w.V), device, 1.0, dt)
        rp = []
        for b in range(w.B):
            r, path = plant_acceptance(logits[b], tokens[b], trees[b], want[b], w.use_root_pred,
                                       w.V, rng)
            rp.append(r)
            planted[b] = path
            want[b] = len(path)
        if w.use_root_pred:
            root_pred = torch.tensor(rp, dtype=torch.int32, device=device)
    h_src = normal_tensor(w.seed, 5, (w.B * w.T if w.per_node else w.B, w.d), device, 1.0, dt)
    W = normal_tensor(w.seed, 6, (w.k, w.d, w.d), device, w.w_std, dt) if with_transfer else None
    return Inputs(
        w=w, q=q, k_cache=k_cache, v_cache=v_cache,
        kv_len=torch.tensor(w.kv_len, dtype=torch.int32, device=device),
        parent=torch.from_numpy(parent).to(device),
        parent_tree=torch.from_numpy(np.ascontiguousarray(trees)).to(device),
        tokens=torch.from_numpy(tokens).to(device),
        logits=logits, root_pred=root_pred, h_src=h_src, W=W,
        want_len=want, planted_path=planted, src_node=src)
