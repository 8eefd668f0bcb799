"""CPU oracle of tree attention over a paged cache (numpy, fp64).

TEST INFRASTRUCTURE ONLY: imported by the tests, never by the product package.

The operation is the one of Section "Tree attention" (a row attends to the whole context, to itself
and to its ancestors in the flattened tree; pseudo rows are ordinary rows of `parent`, Section
"Training stage"); only the storage differs: cache row r of sequence b is row r % page_size of page
block_table[b][r // page_size] of a pool shared by all sequences.  The definition is written out in
its dense-mask form: scores against every logical row, a visibility mask, a softmax, a weighted sum.
"""
from __future__ import annotations

import numpy as np

OK, BAD_TREE, BAD_LEN, BAD_PAGE = 0, 1, 2, 5


def logical_rows(pool, table_b, n_rows):
    """pool [n_pages, Hkv, page_size, D], table_b [max_pages] -> [Hkv, n_rows, D]: the first n_rows
    logical cache rows of one sequence."""
    ps = pool.shape[2]
    r = np.arange(n_rows)
    return np.moveaxis(pool[table_b[r // ps], :, r % ps, :], 0, 1)


def visibility(parent_b, L):
    """[N, L + N] boolean: row r sees the L context rows, itself and its ancestors."""
    N = parent_b.shape[0]
    vis = np.zeros((N, L + N), dtype=bool)
    vis[:, :L] = True
    for r in range(N):
        c = r
        while c >= 0:
            vis[r, L + c] = True
            c = int(parent_b[c])
    return vis


def tree_attention_paged(q, k_pages, v_pages, block_table, kv_len, parent, scale=None):
    """q [B, N, Hq, D]; pools [n_pages, Hkv, page_size, D]; block_table [B, max_pages]; kv_len [B];
    parent [B, N].  Returns (out float64 [B, N, Hq, D], status int32 [B]); rows of sequences with a
    non-zero status are zero."""
    q = np.asarray(q, dtype=np.float64)
    k_pages = np.asarray(k_pages, dtype=np.float64)
    v_pages = np.asarray(v_pages, dtype=np.float64)
    B, N, Hq, D = q.shape
    n_pages, Hkv, ps, _ = k_pages.shape
    g = Hq // Hkv
    max_pages = block_table.shape[1]
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    out = np.zeros_like(q)
    status = np.zeros(B, dtype=np.int32)
    for b in range(B):
        L = int(kv_len[b])
        par = np.asarray(parent[b])
        if any(int(par[r]) < -1 or int(par[r]) >= r for r in range(N)):
            status[b] = BAD_TREE
            continue
        if L < 0 or L + N > max_pages * ps:
            status[b] = BAD_LEN
            continue
        rows = L + N
        used = block_table[b, :(rows + ps - 1) // ps]
        if (used < 0).any() or (used >= n_pages).any():
            status[b] = BAD_PAGE
            continue
        K = logical_rows(k_pages, block_table[b], rows)          # [Hkv, rows, D]
        V = logical_rows(v_pages, block_table[b], rows)
        vis = visibility(par, L)
        for h in range(Hq):
            s = scale * (q[b, :, h, :] @ K[h // g].T)            # [N, rows]
            s = np.where(vis, s, -np.inf)
            w = np.exp(s - s.max(axis=1, keepdims=True))
            w /= w.sum(axis=1, keepdims=True)
            out[b, :, h, :] = w @ V[h // g]
    return out, status


def scatter_to_pages(cache, page_size, order_seed, spare_pages=3, fill=0.0):
    """Input generation for tests: a contiguous cache [B, Hkv, cap, D] (cap a multiple of page_size) cut
    into pages that are placed in a seeded random order in a pool with a few unused pages.  Returns
    (pool [n_pages, Hkv, page_size, D], block_table [B, cap / page_size] int32)."""
    B, Hkv, cap, D = cache.shape
    per = cap // page_size
    n_pages = B * per + spare_pages
    perm = np.random.default_rng(order_seed).permutation(n_pages)[:B * per].astype(np.int32)
    table = perm.reshape(B, per)
    pool = np.full((n_pages, Hkv, page_size, D), fill, dtype=cache.dtype)
    for b in range(B):
        for i in range(per):
            pool[table[b, i]] = cache[b, :, i * page_size:(i + 1) * page_size, :]
    return pool, table


def rope_kv_append_paged(q_in, k_in, v_in, pos, kv_len, block_table, k_pages, v_pages, base=10000.0):
    """The step ahead of attention on a paged cache: q and K rows rotated to their position ids (the rotation
    itself is `rope_oracle.rope`), K and V rows of query row r stored at logical cache row kv_len[b] + r, i.e. at
    row (kv_len[b] + r) % page_size of page block_table[b][(kv_len[b] + r) // page_size].  Copies of the pools
    are returned: (q_out float64, k_pages, v_pages, status).  A sequence that does not fit its table is skipped
    (BAD_LEN); a row whose page entry lies outside the pool is not written and marks the sequence BAD_PAGE."""
    from oracle import rope_oracle
    k_pages = np.array(k_pages, copy=True)
    v_pages = np.array(v_pages, copy=True)
    B, N = pos.shape
    n_pages, Hkv, ps, D = k_pages.shape
    max_pages = block_table.shape[1]
    q_out = np.zeros(np.asarray(q_in).shape, dtype=np.float64)
    status = np.zeros(B, dtype=np.int32)
    for b in range(B):
        L = int(kv_len[b])
        if L < 0 or L + N > max_pages * ps:
            status[b] = BAD_LEN
            continue
        for r in range(N):
            q_out[b, r] = rope_oracle.rope(q_in[b, r], pos[b, r], base)
            row = L + r
            page = int(block_table[b, row // ps])
            if page < 0 or page >= n_pages:
                status[b] = BAD_PAGE
                continue
            k_pages[page, :, row % ps, :] = rope_oracle.rope(k_in[b, r], pos[b, r], base).astype(k_pages.dtype)
            v_pages[page, :, row % ps, :] = v_in[b, r]
    return q_out, k_pages, v_pages, status


def kv_compact_paged(k_pages, v_pages, block_table, n_rows, kv_len, accept_len, accept_path):
    """Compaction on copies of pools [layers, n_pages, Hkv, page_size, D]: for every layer, sequence and
    j < accept_len[b], logical row kv_len[b] + j receives what logical row kv_len[b] + accept_path[b][j] held
    before (all sources read before any row is written).  Returns (k_pages, v_pages, new_kv_len, status)."""
    k_pages = np.array(k_pages, copy=True)
    v_pages = np.array(v_pages, copy=True)
    layers, n_pages, Hkv, ps, D = k_pages.shape
    B, max_pages = block_table.shape
    max_path = accept_path.shape[1]
    new_len = np.array(kv_len, dtype=np.int32, copy=True)
    status = np.zeros(B, dtype=np.int32)
    BAD_PATH = 3
    for b in range(B):
        L, a = int(kv_len[b]), int(accept_len[b])
        if L < 0 or L + n_rows > max_pages * ps:
            status[b] = BAD_LEN
            continue
        path = [int(x) for x in accept_path[b, :max(a, 0)]] if 0 <= a <= max_path else None
        if path is None or a > n_rows or any(p < j or p >= n_rows or (j > 0 and p <= path[j - 1]) for j, p in enumerate(path)):
            status[b] = BAD_PATH
            continue
        rows = [L + p for p in path] + [L + j for j in range(a)]
        pages = [int(block_table[b, r // ps]) for r in rows]
        if any(pg < 0 or pg >= n_pages for pg in pages):
            status[b] = BAD_PAGE
            continue
        for pool in (k_pages, v_pages):
            held = [pool[:, int(block_table[b, (L + p) // ps]), :, (L + p) % ps, :].copy() for p in path]
            for j in range(a):
                pool[:, int(block_table[b, (L + j) // ps]), :, (L + j) % ps, :] = held[j]
        new_len[b] = L + a
    return k_pages, v_pages, new_len, status
