"""Pins of the draft-tree oracle (oracle/draft_oracle.py): the hand-made example, library
top-k, brute force, agreement of the trie statement with the gather statement, and the
property the paper states -- the tree's root paths are exactly the candidate sequences."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import draft_oracle as do


def _golden():
    vals = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "draft_tree_small.txt")):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=")
            vals[k.strip()] = [float(x) for x in v.split()]
    return vals


def test_hand_made_example():
    g = _golden()
    logits = np.array([[g["logits_row1"], g["logits_row2"]]])
    parent = [int(x) for x in g["parent"]]
    rank = [int(x) for x in g["rank"]]
    for fn in (do.draft_tree, do.draft_tree_gather):
        topk, tokens, pos, status = fn(logits, 0, 2, 2, parent, rank, np.array([int(g["root_token"][0])]),
                                       np.array([int(g["base_pos"][0])]))
        assert status.tolist() == [0]
        assert topk[0, 0].tolist() == g["expected_top_row1"] and topk[0, 1].tolist() == g["expected_top_row2"]
        assert tokens[0].tolist() == g["expected_tokens"]
        assert pos[0].tolist() == g["expected_pos"]


def test_top_tokens_against_library_topk_and_brute_force():
    rng = np.random.default_rng(1)
    for V, K in ((7, 3), (50, 8), (1000, 16)):
        x = rng.standard_normal(V)
        top = do.top_tokens(x, K)
        vals, idx = torch.topk(torch.from_numpy(x), K)           # distinct values: indices are unique
        assert top == idx.tolist()
        assert top[0] == int(np.argmax(x))
    # brute force on every permutation of a tiny row with ties
    base = [1.0, 1.0, 0.5, 2.0, 0.5]
    for perm in itertools.permutations(range(5)):
        row = [base[i] for i in perm]
        want = sorted(range(5), key=lambda i: (-row[i], i))[:4]
        assert do.top_tokens(row, 4) == want


def test_top_tokens_ties_nan_and_infinities():
    row = [np.nan, 3.0, 3.0, -np.inf, np.inf, np.nan, 3.0]
    assert do.top_tokens(row, 7) == [4, 1, 2, 6, 3, 0, 5]        # +inf, the 3.0s by index, -inf, then the NaNs by index
    assert do.top_tokens([np.nan] * 4, 2) == [0, 1]
    # rank 0 agrees with the row-argmax rule of the verification oracle (lowest index, NaN never wins)
    from oracle import ht_oracle
    ht_oracle.build()
    rng = np.random.default_rng(2)
    x = np.round(rng.standard_normal((20, 40)) * 2) / 2
    x[3, 5] = np.nan
    assert [do.top_tokens(r, 1)[0] for r in x] == ht_oracle.row_argmax(x.astype(np.float32)).tolist()


def _random_template(rng, T, P, K, has_root):
    parent, rank, depth = [], [], []
    for n in range(T):
        while True:
            p = int(rng.integers(-1, n)) if n else -1
            d = 0 if p < 0 else depth[p] + 1
            if d + (0 if has_root else 1) <= P:
                break
        parent.append(p)
        depth.append(d)
        rank.append(int(rng.integers(0, K)))
    return parent, rank


@pytest.mark.parametrize("has_root", [True, False])
def test_trie_statement_equals_gather_statement_and_paths_are_the_candidates(has_root):
    rng = np.random.default_rng(5)
    for trial in range(30):
        B, P, K, V, T = 2, 3, 4, 30, int(rng.integers(1, 25))
        logits = np.round(rng.standard_normal((B, P + 2, V)) * 3) / 3          # ties happen
        parent, rank = _random_template(rng, T, P, K, has_root)
        root = rng.integers(0, V, B) if has_root else None
        base = rng.integers(0, 100, B)
        a = do.draft_tree(logits, 1, P, K, parent, rank, root, base)
        g = do.draft_tree_gather(logits, 1, P, K, parent, rank, root, base)
        for x, y in zip(a, g):
            assert np.array_equal(x, y)
        depth = do.template_depths(parent)
        for b in range(B):
            # every root path is the candidate its ranks spell out; positions follow the depth
            for n, path in enumerate(do.root_paths(parent, a[1][b])):
                chain = []
                c = n
                while c >= 0:
                    chain.append(c)
                    c = parent[c]
                chain.reverse()
                want = []
                for c in chain:
                    lvl = depth[c] + (0 if has_root else 1)
                    want.append(int(root[b]) if lvl == 0 else do.top_tokens(logits[b, 1 + lvl - 1], K)[rank[c]])
                assert list(path) == want
                assert a[2][b, n] == base[b] + depth[n]


def test_full_cartesian_template_lists_every_candidate_once():
    """Template = all rank tuples of widths (3, 2): its leaves' root paths are the Cartesian product of
    the top lists, and children of one node carry distinct tokens (common ancestors were merged)."""
    rng = np.random.default_rng(7)
    logits = rng.standard_normal((1, 2, 12))
    parent, rank = [], []
    for r1 in range(3):
        parent.append(-1); rank.append(r1)
    for r1 in range(3):
        for r2 in range(2):
            parent.append(r1); rank.append(r2)
    topk, tokens, pos, status = do.draft_tree(logits, 0, 2, 3, parent, rank, None, np.array([10]))
    leaves = [p for p in do.root_paths(parent, tokens[0]) if len(p) == 2]
    want = {(int(topk[0, 0, a]), int(topk[0, 1, b])) for a in range(3) for b in range(2)}
    assert set(leaves) == want and len(leaves) == len(want)
    assert pos[0].tolist() == [10] * 3 + [11] * 6


def test_bad_templates_are_flagged():
    logits = np.zeros((2, 3, 5))
    for parent, rank in (([-1, 1], [0, 0]), ([-1, 0, 1, 2], [0, 0, 0, 0]), ([-1, 0], [0, 9])):
        topk, tokens, pos, status = do.draft_tree(logits, 0, 2, 2, parent, rank, None, np.array([0, 0]))
        assert status.tolist() == [do.BAD_TREE] * 2
        assert (tokens == -1).all()
