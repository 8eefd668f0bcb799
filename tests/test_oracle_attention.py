"""Pins for the oracle's tree attention (CPU only).

Each test checks the oracle against something that is not the oracle: a library causal
SDPA, a closed form, an invariant of the ancestor-only rule (Section "Tree attention";
pseudo rows: Section "Training stage" and the "No masked" ablation).
"""
import numpy as np
import pytest
import torch

from paper_2404_12022_b200 import workloads as wl


def _rand_problem(seed, B=2, N=9, Hq=4, Hkv=2, D=16, L=(5, 11), tree="random"):
    rng = np.random.default_rng(seed)
    cap = max(L) + N + 3
    q = rng.standard_normal((B, N, Hq, D)).astype(np.float32)
    k = rng.standard_normal((B, Hkv, cap, D)).astype(np.float32)
    v = rng.standard_normal((B, Hkv, cap, D)).astype(np.float32)
    parent = np.zeros((B, N), dtype=np.int32)
    for b in range(B):
        for r in range(N):
            if tree == "chain":
                parent[b, r] = r - 1
            elif tree == "roots":
                parent[b, r] = -1
            else:
                parent[b, r] = rng.integers(-1, r) if r > 0 else -1
    return q, k, v, np.array(L[:B], dtype=np.int32), parent


def _path(parent, r):
    out = []
    while r >= 0:
        out.append(r)
        r = parent[r]
    return out[::-1]


def _sdpa_causal_last_rows(qseq, kseq, vseq, scale, n_last):
    """Library causal attention (torch CPU, fp64) over one sequence; returns the last rows."""
    qt = torch.from_numpy(qseq)[None, None].double()
    kt = torch.from_numpy(kseq)[None, None].double()
    vt = torch.from_numpy(vseq)[None, None].double()
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True, scale=scale)
    return o[0, 0, -n_last:].numpy()


def test_two_forms_agree(oracle):
    q, k, v, L, parent = _rand_problem(1)
    a = oracle.tree_attention(q, k, v, L, parent)
    m = oracle.tree_attention_mask_form(q, k, v, L, parent)
    assert np.abs(a - m).max() < 1e-12


def test_each_node_is_causal_attention_over_its_path(oracle):
    """Brute force: gather [context, root..node] and run a library causal attention on it."""
    q, k, v, L, parent = _rand_problem(2, B=2, N=10, Hq=4, Hkv=2, D=8)
    B, N, Hq, D = q.shape
    g = Hq // k.shape[1]
    out = oracle.tree_attention(q, k, v, L, parent)
    scale = 1.0 / np.sqrt(D)
    for b in range(B):
        for r in range(N):
            path = _path(parent[b], r)
            rows = list(range(L[b])) + [L[b] + c for c in path]
            for h in range(Hq):
                kseq = k[b, h // g, rows]
                vseq = v[b, h // g, rows]
                qseq = np.zeros_like(kseq)
                qseq[L[b]:] = q[b, path, h]
                ref = _sdpa_causal_last_rows(qseq, kseq, vseq, scale, 1)[0]
                assert np.abs(out[b, r, h] - ref).max() < 1e-12


def test_chain_is_causal_multi_token_decode(oracle):
    q, k, v, L, parent = _rand_problem(3, tree="chain")
    B, N, Hq, D = q.shape
    g = Hq // k.shape[1]
    out = oracle.tree_attention(q, k, v, L, parent)
    for b in range(B):
        n = L[b] + N
        for h in range(Hq):
            qseq = np.zeros((n, D), dtype=np.float32)
            qseq[L[b]:] = q[b, :, h]
            ref = _sdpa_causal_last_rows(qseq, k[b, h // g, :n], v[b, h // g, :n], 1 / np.sqrt(D), N)
            assert np.abs(out[b, :, h] - ref).max() < 1e-12


def test_independent_roots_are_single_token_decodes(oracle):
    q, k, v, L, parent = _rand_problem(4, tree="roots")
    B, N, Hq, D = q.shape
    g = Hq // k.shape[1]
    out = oracle.tree_attention(q, k, v, L, parent)
    for b in range(B):
        for r in range(N):
            rows = list(range(L[b])) + [L[b] + r]
            for h in range(Hq):
                kk = torch.from_numpy(k[b, h // g, rows]).double()
                vv = torch.from_numpy(v[b, h // g, rows]).double()
                qq = torch.from_numpy(q[b, r, h]).double()
                w = torch.softmax(kk @ qq / np.sqrt(D), dim=0)
                ref = (w[:, None] * vv).sum(0).numpy()
                assert np.abs(out[b, r, h] - ref).max() < 1e-12


def test_closed_form_zero_query_gives_mean_of_visible_values(oracle):
    q, k, v, L, parent = _rand_problem(5)
    q[:] = 0
    out = oracle.tree_attention(q, k, v, L, parent)
    B, N, Hq, D = q.shape
    g = Hq // k.shape[1]
    for b in range(B):
        for r in range(N):
            rows = list(range(L[b])) + [L[b] + c for c in _path(parent[b], r)]
            for h in range(Hq):
                ref = v[b, h // g, rows].astype(np.float64).mean(0)
                assert np.abs(out[b, r, h] - ref).max() < 1e-12


def test_closed_form_constant_values(oracle):
    q, k, v, L, parent = _rand_problem(6)
    const = np.linspace(-1, 1, v.shape[-1]).astype(np.float32)
    v[:] = const
    out = oracle.tree_attention(q, k, v, L, parent)
    assert np.abs(out - const.astype(np.float64)).max() < 1e-12


def test_closed_form_empty_context_single_row(oracle):
    q, k, v, _, _ = _rand_problem(7, B=1, N=1, L=(0,))
    out = oracle.tree_attention(q, k, v, np.array([0], np.int32), np.array([[-1]], np.int32))
    g = q.shape[2] // k.shape[1]
    for h in range(q.shape[2]):
        assert np.abs(out[0, 0, h] - v[0, h // g, 0]).max() < 1e-15


def test_closed_form_two_keys_is_a_sigmoid_blend(oracle):
    """L = 1, one root: out = v0 + sigmoid(scale * q.(k1 - k0)) * (v1 - v0)."""
    q, k, v, _, _ = _rand_problem(8, B=1, N=1, Hq=2, Hkv=2, D=4, L=(1,))
    out = oracle.tree_attention(q, k, v, np.array([1], np.int32), np.array([[-1]], np.int32), scale=0.37)
    for h in range(2):
        z = 0.37 * float(q[0, 0, h].astype(np.float64) @ (k[0, h, 1].astype(np.float64) - k[0, h, 0]))
        s = 1.0 / (1.0 + np.exp(-z))
        ref = v[0, h, 0] + s * (v[0, h, 1].astype(np.float64) - v[0, h, 0])
        assert np.abs(out[0, 0, h] - ref).max() < 1e-12


def test_output_inside_hull_of_visible_values_and_ignores_invisible_rows(oracle):
    q, k, v, L, parent = _rand_problem(9)
    out = oracle.tree_attention(q, k, v, L, parent)
    B, N, Hq, D = q.shape
    g = Hq // k.shape[1]
    for b in range(B):
        for r in range(N):
            rows = list(range(L[b])) + [L[b] + c for c in _path(parent[b], r)]
            for h in range(Hq):
                vis = v[b, h // g, rows]
                assert (out[b, r, h] <= vis.max(0) + 1e-12).all()
                assert (out[b, r, h] >= vis.min(0) - 1e-12).all()
    # scrambling the rows no query may see (other branches, rows past the tree) changes nothing
    k2, v2 = k.copy(), v.copy()
    b, r = 0, N - 1
    seen = set(_path(parent[b], r))
    for c in range(N):
        if c not in seen:
            k2[b, :, L[b] + c] += 100.0
            v2[b, :, L[b] + c] -= 50.0
    k2[b, :, L[b] + N:] = 1e4
    v2[b, :, L[b] + N:] = -1e4
    out2 = oracle.tree_attention(q, k2, v2, L, parent)
    assert np.array_equal(out2[b, r], out[b, r])


def test_gqa_equals_mha_with_repeated_kv_heads(oracle):
    q, k, v, L, parent = _rand_problem(10, Hq=8, Hkv=2)
    out = oracle.tree_attention(q, k, v, L, parent)
    k_rep = np.repeat(k, 4, axis=1)
    v_rep = np.repeat(v, 4, axis=1)
    out_mha = oracle.tree_attention(q, k_rep, v_rep, L, parent)
    assert np.array_equal(out, out_mha)


def test_relabelling_permutes_outputs(oracle):
    """Any ancestor-first renumbering of the tree gives the same outputs, permuted."""
    q, k, v, L, parent = _rand_problem(11, B=1, N=12, L=(7,))
    rng = np.random.default_rng(0)
    N = parent.shape[1]
    # random topological order: repeatedly pick any node whose parent is already placed
    placed, order = set([-1]), []
    while len(order) < N:
        ready = [c for c in range(N) if c not in order and parent[0, c] in placed]
        c = int(rng.choice(ready))
        order.append(c)
        placed.add(c)
    new_of_old = {old: new for new, old in enumerate(order)}
    new_of_old[-1] = -1
    parent2 = np.array([[new_of_old[int(parent[0, old])] for old in order]], dtype=np.int32)
    q2 = q[:, order]
    k2, v2 = k.copy(), v.copy()
    k2[0, :, L[0]:L[0] + N] = k[0, :, [L[0] + o for o in order]].transpose(1, 0, 2)
    v2[0, :, L[0]:L[0] + N] = v[0, :, [L[0] + o for o in order]].transpose(1, 0, 2)
    out = oracle.tree_attention(q, k, v, L, parent)
    out2 = oracle.tree_attention(q2, k2, v2, L, parent2)
    assert np.abs(out2 - out[:, order]).max() < 1e-12


def test_pseudo_rows_see_source_path_and_earlier_pseudo_rows_only(oracle):
    """Pseudo positions hang off their source node as a chain; tree rows never see them."""
    tree = wl.full_binary_tree(3)
    parent = wl.append_pseudo_rows(tree, 4, 3)[None]
    assert parent[0, 15:].tolist() == [4, 15, 16]
    rng = np.random.default_rng(12)
    N, L, D = 18, 6, 8
    q = rng.standard_normal((1, N, 2, D)).astype(np.float32)
    k = rng.standard_normal((1, 2, L + N, D)).astype(np.float32)
    v = rng.standard_normal((1, 2, L + N, D)).astype(np.float32)
    kv_len = np.array([L], np.int32)
    out = oracle.tree_attention(q, k, v, kv_len, parent)
    # second pseudo row == last row of a causal decode over [context, 0, 1, 4, p0, p1]
    rows = list(range(L)) + [L + c for c in (0, 1, 4, 15, 16)]
    for h in range(2):
        qseq = np.zeros((len(rows), D), np.float32)
        qseq[-1] = q[0, 16, h]
        ref = _sdpa_causal_last_rows(qseq, k[0, h, rows], v[0, h, rows], 1 / np.sqrt(D), 1)[0]
        assert np.abs(out[0, 16, h] - ref).max() < 1e-12
    # the tree rows are unchanged when the pseudo rows are dropped
    out_t = oracle.tree_attention(q[:, :15], k, v, kv_len, parent[:, :15])
    assert np.array_equal(out_t, out[:, :15])


def test_selected_rows_match_full(oracle):
    q, k, v, L, parent = _rand_problem(13)
    full = oracle.tree_attention(q, k, v, L, parent)
    sel = np.array([[0, 1, 3], [1, 3, 8], [0, 0, 0]], np.int32)
    part = oracle.tree_attention(q, k, v, L, parent, sel=sel)
    for i, (b, h, r) in enumerate(sel):
        assert np.array_equal(part[i], full[b, r, h])


def test_scale_and_softmax_shift_invariance(oracle):
    """Adding a constant vector c to every key shifts all of a row's scores equally: no change."""
    q, k, v, L, parent = _rand_problem(14, B=1, L=(9,))
    out = oracle.tree_attention(q, k, v, L, parent, scale=0.5)
    # doubling q while halving the scale leaves the scores unchanged (powers of two: exact)
    out2 = oracle.tree_attention(2 * q, k, v, L, parent, scale=0.25)
    assert np.abs(out - out2).max() < 1e-13


def test_illegal_trees_and_lengths_are_rejected(oracle):
    q, k, v, L, parent = _rand_problem(15)
    bad = parent.copy()
    bad[0, 3] = 3
    with pytest.raises(oracle.OracleError) as e:
        oracle.tree_attention(q, k, v, L, bad)
    assert e.value.code == oracle.BAD_TREE
    bad[0, 3] = -2
    with pytest.raises(oracle.OracleError):
        oracle.tree_attention_mask_form(q, k, v, L, bad)
    with pytest.raises(oracle.OracleError) as e:
        oracle.tree_attention(q, k, v, np.array([5, k.shape[2]], np.int32), parent)
    assert e.value.code == oracle.BAD_LEN
