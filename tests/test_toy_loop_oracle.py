"""System pin for the oracle: draft-and-verify rounds reproduce greedy decoding exactly."""
import numpy as np
import pytest

from toy_lm import run_lossless_loop


class OracleOps:
    def __init__(self, oracle):
        self.o = oracle

    def attention(self, q, k_cache, v_cache, kv_len, parent):
        return self.o.tree_attention(q, k_cache, v_cache, kv_len, parent)

    def transfer(self, h, W):
        return self.o.transfer(h, W)

    def verify(self, logits, tokens, parent, root_pred, max_path):
        return self.o.verify_greedy(logits, tokens, parent, root_pred, max_path)

    def compact(self, k_cache, v_cache, N, kv_len, alen, apath):
        k, v, new_len, status = self.o.kv_compact(k_cache, v_cache, N, kv_len, alen, apath)
        assert (status == 0).all()
        return k, v, new_len


@pytest.mark.parametrize("with_root", [True, False])
def test_tree_verify_rounds_equal_greedy_decoding(oracle, with_root):
    rounds = run_lossless_loop(OracleOps(oracle), with_root, seed=3, n_new=24)
    assert rounds < 24          # drafts were accepted along the way, so rounds were saved
