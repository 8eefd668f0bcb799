"""CPU oracle of the draft-tree step (plain Python / numpy, slow on purpose).

TEST INFRASTRUCTURE ONLY: imported by the tests, never by the product package.

What it computes -- Section "Inference stage" and Section "Tree attention": the candidates
for the next positions are sequences of likely tokens, one per future position; "multiple
sequence candidates" are made "into a tree structure by merging their common ancestors", and the
tree is flattened "while preserving the original positional indices of each token"; a
"pre-defined tree structure" fixes which candidates there are.  Here the pre-defined structure
is a template: a parent array whose node n, at depth i below the known next token, stands for
"the rank[n]-th most likely token of future position i" (Section "Setup": the same tree
structure as Medusa, three draft tokens).  Future position i is read from the logits of pseudo
position i (Section "Hidden Transfer": the lm-head decodes the pseudo hidden states).

Two statements of the same result:
  draft_tree          the paper's order: list every candidate sequence the template stands for,
                      merge common prefixes in a trie, flatten, read the tokens off the trie;
  draft_tree_gather   node by node: token = top list of the node's level at the node's rank.
"""
from __future__ import annotations

import math

import numpy as np

OK, BAD_TREE = 0, 1


def top_tokens(row, K):
    """The K most likely entries of one logits row: larger value first, lower index first among
    equals; NaN ranks below everything (NaNs among themselves by index)."""
    def key(i):
        x = float(row[i])
        return (1, 0.0, i) if math.isnan(x) else (0, -x, i)
    order = sorted(range(len(row)), key=key)
    return [int(i) for i in order[:K]]


def template_depths(parent):
    """Depth of every node (top-level nodes: 0), or None when some parent is not an earlier node."""
    depth = []
    for n, p in enumerate(parent):
        if p < -1 or p >= n:
            return None
        depth.append(0 if p < 0 else depth[p] + 1)
    return depth


def _levels(parent, has_root):
    depth = template_depths(parent)
    if depth is None:
        return None, None
    # with a known next token the top-level nodes ARE that token (level 0); without, they are drafts of level 1
    return depth, [d if has_root else d + 1 for d in depth]


def draft_tree(logits, first_row, P, K, parent, rank, root_token, base_pos):
    """logits [B, rows, V]; pseudo position i (1..P) of sequence b is row first_row + i - 1.
    parent, rank [T]; root_token [B] or None; base_pos [B].
    Returns (topk [B, P, K], tokens [B, T], pos [B, T], status [B])."""
    logits = np.asarray(logits, dtype=np.float64)
    B = logits.shape[0]
    T = len(parent)
    has_root = root_token is not None
    topk = np.zeros((B, P, K), np.int32)
    tokens = np.full((B, T), -1, np.int32)
    pos = np.full((B, T), -1, np.int32)
    status = np.zeros(B, np.int32)
    depth, level = _levels(list(parent), has_root)
    bad = depth is None or any(l > P for l in level) or any(l >= 1 and not (0 <= r < K) for l, r in zip(level, rank))
    for b in range(B):
        for i in range(P):
            topk[b, i] = top_tokens(logits[b, first_row + i], K)
        if bad:
            status[b] = BAD_TREE
            continue
        # 1. the candidate sequences: one per template node, the ranks along its root path
        candidates = []
        for n in range(T):
            chain = []
            c = n
            while c >= 0:
                chain.append(c)
                c = parent[c]
            chain.reverse()
            seq = []
            for c in chain:
                if level[c] == 0:
                    seq.append(("root", 0, int(root_token[b])))
                else:
                    seq.append((level[c], int(rank[c]), int(topk[b, level[c] - 1, rank[c]])))
            candidates.append(tuple(seq))
        # 2. merge common ancestors: a trie; two candidates share a node while their steps agree
        trie = {}
        for seq in candidates:
            kids = trie
            for step in seq:
                node = kids.setdefault(step[:-1], {"token": step[-1], "kids": {}})
                assert node["token"] == step[-1]               # the same step always means the same token
                kids = node["kids"]
        # 3. flatten in template order: node n is where its own candidate ends in the merged tree
        for n, seq in enumerate(candidates):
            kids, node = trie, None
            for step in seq:
                node = kids[step[:-1]]
                kids = node["kids"]
            tokens[b, n] = node["token"]
            pos[b, n] = int(base_pos[b]) + depth[n]
    return topk, tokens, pos, status


def draft_tree_gather(logits, first_row, P, K, parent, rank, root_token, base_pos):
    """Second statement: no candidates, no trie."""
    logits = np.asarray(logits, dtype=np.float64)
    B = logits.shape[0]
    T = len(parent)
    has_root = root_token is not None
    topk = np.zeros((B, P, K), np.int32)
    tokens = np.full((B, T), -1, np.int32)
    pos = np.full((B, T), -1, np.int32)
    status = np.zeros(B, np.int32)
    depth, level = _levels(list(parent), has_root)
    bad = depth is None or any(l > P for l in level) or any(l >= 1 and not (0 <= r < K) for l, r in zip(level, rank))
    for b in range(B):
        for i in range(P):
            topk[b, i] = top_tokens(logits[b, first_row + i], K)
        if bad:
            status[b] = BAD_TREE
            continue
        for n in range(T):
            tokens[b, n] = int(root_token[b]) if level[n] == 0 else topk[b, level[n] - 1, rank[n]]
            pos[b, n] = int(base_pos[b]) + depth[n]
    return topk, tokens, pos, status


def root_paths(parent, tokens_b):
    """Every root-to-node token sequence of a flattened tree (for the tests)."""
    out = []
    for n in range(len(parent)):
        seq = []
        c = n
        while c >= 0:
            seq.append(int(tokens_b[c]))
            c = parent[c]
        out.append(tuple(reversed(seq)))
    return out
