"""Host-side checks of the synthetic input generators and of config 1 through the oracle."""
import dataclasses

import numpy as np
import torch

from paper_2404_12022_b200 import workloads as wl


def test_hashed_normal_is_sliceable_and_standard():
    full = wl.hashed_normal(7, 3, 0, 200000)
    part = wl.hashed_normal(7, 3, 1234, 5000)
    assert torch.equal(full[1234:6234], part)
    assert abs(float(full.mean())) < 0.01 and abs(float(full.std()) - 1.0) < 0.01
    assert float(full.abs().max()) < wl.PLANTED_LOGIT
    other = wl.hashed_normal(7, 4, 0, 1000)
    assert not torch.equal(full[:1000], other)
    big = wl.hashed_normal(7, 3, (1 << 33) + 5, 100)       # indices beyond 32 bits still work
    assert big.isfinite().all() and not torch.equal(big, full[5:105])
    # chunking does not change the values
    assert torch.equal(wl.hashed_normal(7, 3, 0, 5000, chunk=777), full[:5000])


def test_tree_shapes_of_the_configs():
    assert wl.full_binary_tree(3).tolist() == [-1, 0, 0, 1, 1, 2, 2, 3, 3, 4, 4, 5, 5, 6, 6]
    f = wl.level_tree([4, 12, 24, 48])
    assert len(f) == 88 and (f[:4] == -1).all() and f[4:16].tolist() == [0] * 3 + [1] * 3 + [2] * 3 + [3] * 3
    assert wl.node_depths(f).max() == 4
    c = wl.truncated_cartesian_tree([8, 4, 2], 64)
    assert len(c) == 64 and c[0] == -1 and (c[1:9] == 0).all() and wl.node_depths(c).max() == 4
    rng = np.random.Generator(np.random.Philox(1))
    r = wl.random_depth_tree(256, 6, rng)
    assert all(r[i] < i for i in range(256)) and wl.node_depths(r).max() <= 7
    p = wl.append_pseudo_rows(f, 5, 3)
    assert p[88:].tolist() == [5, 88, 89]


def test_planted_acceptance_is_what_the_oracle_finds(oracle):
    for want in (0, 1, 2, 3, 4):
        w = dataclasses.replace(wl.config_c2(), V=500, d=64, kv_len=[16], want_len=[want])
        inp = wl.make_inputs(w)
        pred, alen, apath, nxt, status = oracle.verify_greedy(
            inp.logits.float().numpy(), inp.tokens.numpy(), inp.parent.numpy(),
            inp.root_pred.numpy(), w.max_path)
        assert alen[0] == want == inp.want_len[0]
        assert apath[0, :want].tolist() == inp.planted_path[0]


def test_config_c1_through_the_oracle(oracle):
    """Config 1 end to end on the CPU: runs in seconds, accepted paths of 2 and of 3 nodes."""
    for want in (2, 3):
        w = wl.config_c1(want)
        inp = wl.make_inputs(w)
        assert inp.parent.shape == (1, 18) and inp.q[0].shape == (1, 18, 4, 64)
        out = oracle.tree_attention(inp.q[0].numpy(), inp.k_cache[0].numpy(), inp.v_cache[0].numpy(),
                                    inp.kv_len.numpy(), inp.parent.numpy())
        out_m = oracle.tree_attention_mask_form(inp.q[0].numpy(), inp.k_cache[0].numpy(),
                                                inp.v_cache[0].numpy(), inp.kv_len.numpy(),
                                                inp.parent.numpy())
        assert np.abs(out - out_m).max() < 1e-12
        pseudo = oracle.transfer(inp.h_src.numpy(), inp.W.numpy())
        assert pseudo.shape == (1, 3, 256)
        pred, alen, apath, nxt, status = oracle.verify_greedy(
            inp.logits.numpy(), inp.tokens.numpy(), inp.parent.numpy(), None, w.max_path)
        assert alen[0] == want and apath[0, 0] == 0
        k2, v2, new_len, st = oracle.kv_compact(inp.k_cache.numpy(), inp.v_cache.numpy(), w.N,
                                                inp.kv_len.numpy(), alen, apath)
        assert new_len[0] == 128 + want and st[0] == 0


def test_config_shapes():
    c3 = wl.config_c3()
    assert (c3.N, c3.rows_at_layer(15), c3.rows_at_layer(16), c3.cap) == (91, 88, 91, 4224)
    c4 = wl.config_c4()
    assert len(c4.kv_len) == 8 and min(c4.kv_len) >= 512 and max(c4.kv_len) <= 8192 and c4.N == 68
    assert len(wl.c5_points()) == 48
    c5 = wl.config_c5(32768, 256, 16)
    assert c5.N == 259 and c5.Hq // c5.Hkv == 8
    s = wl.make_structure(wl.config_c3(B=4))
    parent, want = s[1], s[4]
    assert parent.shape == (4, 91) and all(0 <= x <= 4 for x in want)
    assert (parent[0, :88] == wl.level_tree([4, 12, 24, 48])).all()
    assert not (parent[1, :88] == parent[0, :88]).all()
