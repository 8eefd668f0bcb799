"""Pins of the paged-cache attention oracle: against the contiguous oracle (itself pinned elsewhere), against a
brute-force evaluation element by element, and the invariances the storage scheme must have."""
import numpy as np
import pytest

from oracle import ht_oracle, paged_oracle


def case(seed, B=2, N=5, Hq=4, Hkv=2, D=8, ps=4, per=6, lens=(9, 14)):
    rng = np.random.default_rng(seed)
    cap = ps * per
    q = rng.standard_normal((B, N, Hq, D)).astype(np.float32)
    k = rng.standard_normal((B, Hkv, cap, D)).astype(np.float32)
    v = rng.standard_normal((B, Hkv, cap, D)).astype(np.float32)
    parent = np.stack([np.array([-1] + [rng.integers(-1, r) for r in range(1, N)], np.int32) for _ in range(B)])
    return q, k, v, np.array(lens, np.int32), parent, ps


def test_identity_table_is_the_contiguous_oracle():
    q, k, v, kv_len, parent, ps = case(1)
    B, Hkv, cap, D = k.shape
    per = cap // ps
    # pool = the contiguous cache cut in order: page b * per + i holds rows [i ps, (i + 1) ps) of sequence b
    pool_k = k.reshape(B, Hkv, per, ps, D).transpose(0, 2, 1, 3, 4).reshape(B * per, Hkv, ps, D)
    pool_v = v.reshape(B, Hkv, per, ps, D).transpose(0, 2, 1, 3, 4).reshape(B * per, Hkv, ps, D)
    table = np.arange(B * per, dtype=np.int32).reshape(B, per)
    got, status = paged_oracle.tree_attention_paged(q, pool_k, pool_v, table, kv_len, parent)
    assert status.tolist() == [0, 0]
    want = ht_oracle.tree_attention(q, k, v, kv_len, parent)
    assert np.abs(got - want).max() < 1e-12


@pytest.mark.parametrize("seed", [2, 3])
def test_any_placement_of_the_pages_gives_the_same_result(seed):
    q, k, v, kv_len, parent, ps = case(seed)
    want = ht_oracle.tree_attention(q, k, v, kv_len, parent)
    for order in (10, 11):
        pool_k, table = paged_oracle.scatter_to_pages(k, ps, order, fill=np.nan)
        pool_v, table_v = paged_oracle.scatter_to_pages(v, ps, order, fill=np.nan)
        assert np.array_equal(table, table_v)
        got, status = paged_oracle.tree_attention_paged(q, pool_k, pool_v, table, kv_len, parent)
        assert status.tolist() == [0, 0]
        assert np.abs(got - want).max() < 1e-12


def test_brute_force_element_by_element():
    q, k, v, kv_len, parent, ps = case(4, B=1, N=4, Hq=2, Hkv=1, D=4, ps=2, per=5, lens=(5,))
    pool_k, table = paged_oracle.scatter_to_pages(k, ps, 12)
    pool_v, _ = paged_oracle.scatter_to_pages(v, ps, 12)
    got, _ = paged_oracle.tree_attention_paged(q, pool_k, pool_v, table, kv_len, parent)
    L, N, D = 5, 4, 4
    for r in range(N):
        keys = list(range(L))
        c = r
        chain = []
        while c >= 0:
            chain.append(L + c)
            c = int(parent[0, c])
        keys += sorted(chain)
        for h in range(2):
            scores = []
            for key in keys:
                page, off = int(table[0, key // ps]), key % ps
                scores.append(sum(float(q[0, r, h, x]) * float(pool_k[page, 0, off, x]) for x in range(D)) / 2.0)
            m = max(scores)
            w = [np.exp(s - m) for s in scores]
            for x in range(D):
                acc = 0.0
                for wi, key in zip(w, keys):
                    acc += wi * float(pool_v[int(table[0, key // ps]), 0, key % ps, x])
                assert abs(acc / sum(w) - got[0, r, h, x]) < 1e-12


def test_table_entries_past_the_last_used_page_are_free_and_needed_ones_are_checked():
    q, k, v, kv_len, parent, ps = case(5)
    pool_k, table = paged_oracle.scatter_to_pages(k, ps, 13)
    pool_v, _ = paged_oracle.scatter_to_pages(v, ps, 13)
    want, _ = paged_oracle.tree_attention_paged(q, pool_k, pool_v, table, kv_len, parent)
    N = q.shape[1]
    t2 = table.copy()
    for b in range(2):
        t2[b, (int(kv_len[b]) + N + ps - 1) // ps:] = -7
    got, status = paged_oracle.tree_attention_paged(q, pool_k, pool_v, t2, kv_len, parent)
    assert status.tolist() == [0, 0] and np.array_equal(got, want)
    t3 = table.copy()
    t3[1, 0] = pool_k.shape[0]                       # first page of sequence 1: outside the pool
    got, status = paged_oracle.tree_attention_paged(q, pool_k, pool_v, t3, kv_len, parent)
    assert status.tolist() == [0, paged_oracle.BAD_PAGE]
    assert np.array_equal(got[0], want[0]) and not got[1].any()


def test_length_and_tree_checks():
    q, k, v, kv_len, parent, ps = case(6)
    pool_k, table = paged_oracle.scatter_to_pages(k, ps, 14)
    pool_v, _ = paged_oracle.scatter_to_pages(v, ps, 14)
    bad_len = kv_len.copy()
    bad_len[0] = ps * table.shape[1] - q.shape[1] + 1
    _, status = paged_oracle.tree_attention_paged(q, pool_k, pool_v, table, bad_len, parent)
    assert status.tolist() == [paged_oracle.BAD_LEN, 0]
    bad_tree = parent.copy()
    bad_tree[1, 2] = 2
    _, status = paged_oracle.tree_attention_paged(q, pool_k, pool_v, table, kv_len, bad_tree)
    assert status.tolist() == [0, paged_oracle.BAD_TREE]


def _gather(pool, table, cap):
    """[n_pages, Hkv, ps, D] + table [B, per] -> contiguous [B, Hkv, cap, D] (pages that are not allocated read as 0)."""
    B = table.shape[0]
    ps = pool.shape[2]
    out = np.zeros((B, pool.shape[1], cap, pool.shape[3]), pool.dtype)
    for b in range(B):
        for i in range(cap // ps):
            if 0 <= table[b, i] < pool.shape[0]:
                out[b, :, i * ps:(i + 1) * ps] = pool[table[b, i]]
    return out


def test_paged_append_places_rows_where_the_contiguous_append_does():
    from oracle import rope_oracle
    rng = np.random.default_rng(7)
    B, N, Hq, Hkv, D, ps, per = 2, 5, 4, 2, 8, 4, 6
    cap = ps * per
    k = rng.standard_normal((B, Hkv, cap, D))
    v = rng.standard_normal((B, Hkv, cap, D))
    q_in = rng.standard_normal((B, N, Hq, D))
    k_in = rng.standard_normal((B, N, Hkv, D))
    v_in = rng.standard_normal((B, N, Hkv, D))
    kv_len = np.array([3, 17], np.int32)
    pos = (kv_len[:, None] + rng.integers(0, 4, (B, N))).astype(np.int32)
    pool_k, table = paged_oracle.scatter_to_pages(k, ps, 21)
    pool_v, _ = paged_oracle.scatter_to_pages(v, ps, 21)
    q1, pk, pv, st = paged_oracle.rope_kv_append_paged(q_in, k_in, v_in, pos, kv_len, table, pool_k, pool_v)
    q2, ck, cv, st2 = rope_oracle.rope_kv_append(q_in, k_in, v_in, pos, kv_len, k, v)
    assert st.tolist() == [0, 0] and list(st2) == [0, 0]
    assert np.array_equal(q1, q2)
    assert np.array_equal(_gather(pk, table, cap), ck) and np.array_equal(_gather(pv, table, cap), cv)
    # a row whose page is outside the pool is not written; the rest of the sequence is
    t2 = table.copy()
    t2[1, (17 + 4) // ps] = -1
    _, pk2, _, st3 = paged_oracle.rope_kv_append_paged(q_in, k_in, v_in, pos, kv_len, t2, pool_k, pool_v)
    assert st3.tolist() == [0, paged_oracle.BAD_PAGE]
    changed = np.argwhere((pk2 != pool_k).any(axis=(1, 3)))
    assert {(int(p), int(r)) for p, r in changed} == {(int(table[b, (kv_len[b] + r) // ps]), int((kv_len[b] + r) % ps))
                                                      for b in range(B) for r in range(N) if not (b == 1 and (17 + r) // ps == 5)}


def test_paged_compaction_is_the_contiguous_compaction_seen_through_the_table():
    rng = np.random.default_rng(8)
    layers, B, Hkv, D, ps, per, N = 2, 3, 2, 8, 4, 5, 7
    cap = ps * per
    k = rng.integers(0, 250, (layers, B, Hkv, cap, D)).astype(np.uint8)
    v = rng.integers(0, 250, (layers, B, Hkv, cap, D)).astype(np.uint8)
    kv_len = np.array([2, 9, 13], np.int32)
    accept_len = np.array([3, 0, 4], np.int32)
    accept_path = np.array([[0, 2, 5, -1], [-1, -1, -1, -1], [1, 2, 4, 6]], np.int32)
    pools_k, pools_v = [], []
    for l in range(layers):
        pk, table = paged_oracle.scatter_to_pages(k[l], ps, 31)
        pv, _ = paged_oracle.scatter_to_pages(v[l], ps, 31)
        pools_k.append(pk)
        pools_v.append(pv)
    pools_k, pools_v = np.stack(pools_k), np.stack(pools_v)
    gk, gv, new_len, st = paged_oracle.kv_compact_paged(pools_k, pools_v, table, N, kv_len, accept_len, accept_path)
    ck, cv, want_len, want_st = ht_oracle.kv_compact(k, v, N, kv_len, accept_len, accept_path)
    assert st.tolist() == list(want_st) == [0, 0, 0] and new_len.tolist() == list(want_len)
    for l in range(layers):
        for b in range(B):
            keep = int(new_len[b])          # rows at or beyond the new length are unspecified
            assert np.array_equal(_gather(gk[l], table, cap)[b, :, :keep], ck[l, b, :, :keep])
            assert np.array_equal(_gather(gv[l], table, cap)[b, :, :keep], cv[l, b, :, :keep])
    # a path that is not increasing, a length that does not fit, a page outside the pool
    bad = accept_path.copy()
    bad[0] = [2, 1, 5, -1]
    assert paged_oracle.kv_compact_paged(pools_k, pools_v, table, N, kv_len, accept_len, bad)[3].tolist() == [3, 0, 0]
    assert paged_oracle.kv_compact_paged(pools_k, pools_v, table, N, np.array([2, 14, 13], np.int32), accept_len,
                                         accept_path)[3].tolist() == [0, paged_oracle.BAD_LEN, 0]
    t2 = table.copy()
    t2[2, (13 + 6) // ps] = 99
    out = paged_oracle.kv_compact_paged(pools_k, pools_v, t2, N, kv_len, accept_len, accept_path)
    assert out[3].tolist() == [0, 0, paged_oracle.BAD_PAGE] and out[2].tolist() == [5, 9, 13]
