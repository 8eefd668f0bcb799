"""CPU oracle of the step ahead of attention: rotary position embedding at the tree's position
ids and placement of the new K / V rows behind the context (numpy, fp64).

TEST INFRASTRUCTURE ONLY: imported by the tests, never by the product package.

The paper keeps "the original positional indices of each token" when the tree is flattened
(Section "Tree attention") and gives a pseudo state of step i the position id j + i (Section
"Training stage"); its models are LLaMA-2 / Vicuna (Section "Setup"), whose position encoding is
the rotary embedding in the half-split pairing: feature i is paired with feature i + D/2 and the
pair is rotated by the angle pos * base^(-2i/D).  The rows' K and V then sit at cache rows
kv_len[b] + r, which is where the attention entry point expects them.
"""
from __future__ import annotations

import numpy as np

OK, BAD_LEN = 0, 2


def rope(x, pos, base=10000.0):
    """x [..., D] rotated to position `pos` (scalar or broadcastable to x.shape[:-1])."""
    x = np.asarray(x, dtype=np.float64)
    D = x.shape[-1]
    half = D // 2
    i = np.arange(half, dtype=np.float64)
    theta = base ** (-2.0 * i / D)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * theta
    c, s = np.cos(ang), np.sin(ang)
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def rope_kv_append(q_in, k_in, v_in, pos, kv_len, k_cache, v_cache, base=10000.0):
    """q_in [B, N, Hq, D], k_in / v_in [B, N, Hkv, D], pos [B, N], kv_len [B]; caches [B, Hkv, cap, D]
    (copies are returned).  Returns (q_out fp64, k_cache, v_cache, status)."""
    q_in = np.asarray(q_in, dtype=np.float64)
    k_in = np.asarray(k_in, dtype=np.float64)
    B, N = pos.shape
    cap = k_cache.shape[2]
    q_out = np.zeros_like(q_in)
    kc, vc = np.array(k_cache, dtype=np.float64), np.array(v_cache, dtype=np.float64)
    status = np.zeros(B, np.int32)
    for b in range(B):
        L = int(kv_len[b])
        if L < 0 or L + N > cap:
            status[b] = BAD_LEN
            continue
        for r in range(N):
            q_out[b, r] = rope(q_in[b, r], float(pos[b, r]), base)
            kc[b, :, L + r] = rope(k_in[b, r], float(pos[b, r]), base)
            vc[b, :, L + r] = v_in[b, r]
    return q_out, kc, vc, status
