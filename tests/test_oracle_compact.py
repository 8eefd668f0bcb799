"""Pins for the oracle's KV compaction (accepted-path rows moved behind the context)."""
import numpy as np


def _caches(seed, layers=3, B=2, Hkv=2, cap=24, D=4):
    rng = np.random.default_rng(seed)
    k = rng.integers(0, 65535, (layers, B, Hkv, cap, D)).astype(np.uint16)
    v = rng.integers(0, 65535, (layers, B, Hkv, cap, D)).astype(np.uint16)
    return k, v


def test_matches_fancy_index_definition_with_aliasing_path(oracle):
    k, v = _caches(0)
    N = 8
    kv_len = np.array([5, 9], np.int32)
    alen = np.array([3, 2], np.int32)
    path = np.array([[0, 2, 5, -1], [1, 7, -1, -1]], np.int32)   # row L+2 is read and overwritten
    k2, v2, new_len, status = oracle.kv_compact(k, v, N, kv_len, alen, path)
    assert (status == 0).all() and new_len.tolist() == [8, 11]
    for old, new in ((k, k2), (v, v2)):
        ref = old.copy()
        for b in range(2):
            for j in range(alen[b]):
                ref[:, b, :, kv_len[b] + j] = old[:, b, :, kv_len[b] + path[b, j]]
        assert np.array_equal(new, ref)
        for b in range(2):
            assert np.array_equal(new[:, b, :, :kv_len[b]], old[:, b, :, :kv_len[b]])


def test_identity_path_and_empty_acceptance_change_nothing(oracle):
    k, v = _caches(1)
    kv_len = np.array([4, 4], np.int32)
    path = np.array([[0, 1, 2], [-1, -1, -1]], np.int32)
    k2, v2, new_len, status = oracle.kv_compact(k, v, 6, kv_len, np.array([3, 0], np.int32), path)
    assert np.array_equal(k, k2) and np.array_equal(v, v2)
    assert new_len.tolist() == [7, 4] and (status == 0).all()


def test_bad_paths_are_flagged_and_skipped(oracle):
    k, v = _caches(2)
    kv_len = np.array([4, 20], np.int32)
    path = np.array([[2, 1, -1], [0, 1, 2]], np.int32)          # not increasing; does not fit in cap
    k2, v2, new_len, status = oracle.kv_compact(k, v, 6, kv_len, np.array([2, 3], np.int32), path)
    assert status.tolist() == [oracle.BAD_PATH, oracle.BAD_LEN]
    assert np.array_equal(k, k2) and np.array_equal(v, v2) and new_len.tolist() == [4, 20]


def test_element_width_is_respected(oracle):
    rng = np.random.default_rng(3)
    k = rng.standard_normal((1, 1, 1, 10, 3)).astype(np.float32)
    v = rng.standard_normal((1, 1, 1, 10, 3)).astype(np.float32)
    k2, v2, _, _ = oracle.kv_compact(k, v, 5, np.array([2], np.int32), np.array([2], np.int32),
                                      np.array([[1, 4]], np.int32))
    assert np.array_equal(k2[0, 0, 0, 2], k[0, 0, 0, 3]) and np.array_equal(k2[0, 0, 0, 3], k[0, 0, 0, 6])
    assert np.array_equal(v2[0, 0, 0, 3], v[0, 0, 0, 6])
