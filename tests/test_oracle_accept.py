"""Pins for the oracle's greedy verification (Fig. 2 caption; Sections "Inference stage", "Setup").

The reference here is a third, recursive statement written in the test: walk down from
the context, at every step keeping only children that carry the token greedy decoding
would emit next.  It is compared with both oracle forms exhaustively on small trees.
"""
import itertools

import numpy as np
import pytest


def _descend(tokens, parent, pred, root_pred, T):
    """Longest greedy-consistent root path by recursion; ties -> smallest terminal index."""
    kids = {}
    for c in range(T):
        kids.setdefault(int(parent[c]), []).append(c)

    def best_from(node, expected):
        # returns (length, terminal) of the best path continuing below `node`
        best = (0, -1)
        for c in kids.get(node, []):
            if expected is not None and tokens[c] != expected:
                continue
            ln, term = best_from(c, pred[c])
            ln, term = ln + 1, (c if term < 0 else term)
            if ln > best[0] or (ln == best[0] and term < best[1]):
                best = (ln, term)
        return best

    ln, term = best_from(-1, root_pred)
    path = []
    c = term
    while c >= 0:
        path.append(c)
        c = int(parent[c])
    path.reverse()
    nxt = pred[term] if ln > 0 else (root_pred if root_pred is not None else -1)
    return ln, path, nxt


def _all_trees(n):
    """Every parent array with parent[r] in [-1, r)."""
    ranges = [range(-1, r) for r in range(n)]
    return itertools.product(*ranges)


@pytest.mark.parametrize("with_root_pred", [False, True])
def test_exhaustive_small_trees(oracle, with_root_pred):
    """All trees with up to 5 nodes x all token / prediction assignments over 2 symbols (plus
    a seeded sample for 6 nodes over 3 symbols)."""
    cases = []
    for n in range(1, 6):
        for par in _all_trees(n):
            for tok in itertools.product(range(2), repeat=n):
                for prd in itertools.product(range(2), repeat=n):
                    cases.append((par, tok, prd))
    rng = np.random.default_rng(0)
    trees6 = list(_all_trees(6))
    for _ in range(4000):
        par = trees6[int(rng.integers(len(trees6)))]
        cases.append((par, tuple(rng.integers(0, 3, 6)), tuple(rng.integers(0, 3, 6))))
    # run them through the oracle in batches of equal size
    by_n = {}
    for c in cases:
        by_n.setdefault(len(c[0]), []).append(c)
    total = 0
    for n, group in by_n.items():
        par = np.array([g[0] for g in group], np.int32)
        tok = np.array([g[1] for g in group], np.int32)
        prd = np.array([g[2] for g in group], np.int32)
        rp = (np.arange(len(group)) % 2).astype(np.int32) if with_root_pred else None
        res_e = oracle.accept_enumerate(tok, par, prd, rp, 8)
        res_s = oracle.accept_scan(tok, par, prd, rp, 8)
        for a, b in zip(res_e, res_s):
            assert np.array_equal(a, b)
        alen, apath, nxt, status = res_e
        assert (status == 0).all()
        for i in range(len(group)):
            ln, path, want_next = _descend(tok[i], par[i], prd[i], None if rp is None else int(rp[i]), n)
            assert alen[i] == ln
            assert apath[i, :ln].tolist() == path and (apath[i, ln:] == -1).all()
            assert nxt[i] == want_next
            total += 1
    assert total > 30000


def test_never_accepts_a_rejected_token_and_is_maximal(oracle):
    rng = np.random.default_rng(1)
    B, T, P = 64, 40, 3
    N = T + P
    par = np.full((B, N), -1, np.int32)
    for b in range(B):
        for r in range(1, N):
            par[b, r] = rng.integers(-1, r)
    tok = rng.integers(0, 4, (B, T)).astype(np.int32)
    prd = rng.integers(0, 4, (B, N)).astype(np.int32)
    rp = rng.integers(0, 4, B).astype(np.int32)
    alen, apath, nxt, status = oracle.accept_enumerate(tok, par, prd, rp, 16)
    for b in range(B):
        path = apath[b, :alen[b]]
        prev = -1
        for c in path:
            assert par[b, c] == prev
            want = rp[b] if prev < 0 else prd[b, prev]
            assert tok[b, c] == want                      # nothing the argmax rejects is accepted
            prev = c
        last = prev
        expected = rp[b] if last < 0 else prd[b, last]
        for c in range(T):                                 # and the path cannot be extended
            if par[b, c] == last:
                assert tok[b, c] != expected
        assert nxt[b] == expected


def test_chain_all_match_none_match_and_unconditional_root(oracle):
    T = 6
    par = np.arange(-1, T - 1, dtype=np.int32)[None]
    prd = np.array([[10, 11, 12, 13, 14, 15]], np.int32)
    tok = np.array([[9, 10, 11, 12, 13, 14]], np.int32)
    alen, apath, nxt, _ = oracle.accept_scan(tok, par, prd, np.array([9], np.int32), 8)
    assert alen[0] == T and apath[0, :T].tolist() == list(range(T)) and nxt[0] == 15
    alen, _, nxt, _ = oracle.accept_scan(tok, par, prd, np.array([7], np.int32), 8)
    assert alen[0] == 0 and nxt[0] == 7
    tok2 = np.array([[9, 99, 11, 12, 13, 14]], np.int32)
    alen, apath, nxt, _ = oracle.accept_scan(tok2, par, prd, None, 8)
    assert alen[0] == 1 and apath[0, 0] == 0 and nxt[0] == 10      # root taken as known-correct
    alen, _, _, status = oracle.accept_scan(tok, par, prd, np.array([9], np.int32), 4)
    assert status[0] == oracle.PATH_TOO_LONG and alen[0] == 0


def test_ties_between_duplicate_siblings_pick_the_smallest_terminal(oracle):
    par = np.array([[-1, 0, 0, 1, 2]], np.int32)
    tok = np.array([[5, 6, 6, 7, 7]], np.int32)
    prd = np.array([[6, 7, 7, 0, 0]], np.int32)
    alen, apath, nxt, _ = oracle.accept_enumerate(tok, par, prd, np.array([5], np.int32), 4)
    assert alen[0] == 3 and apath[0, :3].tolist() == [0, 1, 3]


def test_row_argmax_ties_nan_and_library_agreement(oracle):
    rng = np.random.default_rng(2)
    x = np.round(rng.standard_normal((50, 300)) * 2).astype(np.float32)   # many exact ties
    pred = oracle.row_argmax(x)
    assert np.array_equal(pred, np.argmax(x, axis=1))                      # numpy: first maximum
    y = x.copy()
    y[0, :] = np.nan
    y[1, 5] = np.nan
    y[2, 0] = np.inf
    y[3, :] = -np.inf
    pred = oracle.row_argmax(y)
    assert pred[0] == 0
    assert pred[1] == np.nanargmax(y[1])
    assert pred[2] == 0 and pred[3] == 0
