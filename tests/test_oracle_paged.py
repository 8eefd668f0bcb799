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
