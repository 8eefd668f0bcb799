"""The C-ABI library loads, exports what include/ht.h declares, and rejects bad arguments on
the host before anything is launched (no GPU needed for any of this)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2404_12022_b200 import build, binding
    build.build()
    return binding.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "ht.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ht_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2404_12022_b200 import binding
    names = _declared()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None
    assert lib.ht_version() >= 100


def test_host_side_rejections(lib):
    from paper_2404_12022_b200 import binding as hb
    buf = (ctypes.c_char * 4096)()
    base = ctypes.addressof(buf)
    p = (base + 255) // 256 * 256          # a 16-byte aligned host address: never dereferenced here
    assert lib.ht_transfer(None, p, p, 1, 1, 8, hb.HT_BF16, None) == hb.HT_ERR_INVALID_ARG
    assert b"NULL" in lib.ht_last_error_string()
    assert lib.ht_transfer(p + 2, p, p, 1, 1, 8, hb.HT_BF16, None) == hb.HT_ERR_INVALID_ARG
    assert lib.ht_transfer(p, p, p, 1, 1, 12, hb.HT_BF16, None) == hb.HT_ERR_UNSUPPORTED
    assert lib.ht_transfer(p, p, p, 1, 1, 8, 7, None) == hb.HT_ERR_INVALID_ARG
    assert lib.ht_transfer(p, p, p, 0, 3, 8, hb.HT_F32, None) == hb.HT_OK      # empty batch: no-op

    d = hb.AttnDesc(1, 4, 6, 4, 128, 64, hb.HT_F16, 0.0, 0, 0, 0, 0)           # Hq % Hkv != 0
    assert lib.ht_tree_attention(ctypes.byref(d), p, p, p, p, p, p, None, 0, p, None) == hb.HT_ERR_INVALID_ARG
    d = hb.AttnDesc(1, 4, 4, 4, 96, 64, hb.HT_F16, 0.0, 0, 0, 0, 0)            # head size not built
    assert lib.ht_tree_attention(ctypes.byref(d), p, p, p, p, p, p, None, 0, p, None) == hb.HT_ERR_UNSUPPORTED
    d = hb.AttnDesc(1, 100, 4, 4, 128, 64, hb.HT_F16, 0.0, 0, 0, 0, 0)         # N > cap
    assert lib.ht_tree_attention(ctypes.byref(d), p, p, p, p, p, p, None, 0, p, None) == hb.HT_ERR_INVALID_ARG
    d = hb.AttnDesc(4, 91, 32, 32, 128, 4224, hb.HT_BF16, 0.0, 0, 0, 4, 0)     # needs a workspace
    need = lib.ht_tree_attention_workspace(ctypes.byref(d))
    assert need > 0 and need % 256 == 0
    assert lib.ht_tree_attention(ctypes.byref(d), p, p, p, p, p, p, p, need - 16, p, None) == hb.HT_ERR_WORKSPACE
    assert lib.ht_tree_attention(ctypes.byref(d), p, p, p, p, p, p, None, 0, p, None) == hb.HT_ERR_WORKSPACE
    d = hb.AttnDesc(0, 91, 32, 32, 128, 4224, hb.HT_BF16, 0.0, 0, 0, 0, 0)     # empty batch
    assert lib.ht_tree_attention(ctypes.byref(d), None, None, None, None, None, None, None, 0, None, None) == hb.HT_OK

    assert lib.ht_verify_greedy(p, hb.HT_F16, p, p, None, 1, 4, 5, 100, 8, p, p, p, p, p, None) == hb.HT_ERR_INVALID_ARG
    assert lib.ht_verify_greedy(p, hb.HT_F16, p, p, None, 1, 4, 3, 100, 8, None, p, p, p, p, None) == hb.HT_ERR_INVALID_ARG
    assert lib.ht_verify_greedy(p, hb.HT_F16, p, p, None, 1, 4, 3, 100, 0, p, p, p, p, p, None) == hb.HT_ERR_INVALID_ARG

    assert lib.ht_verify_greedy(p, hb.HT_F16, p, p, None, 1, 4, 3, 100, 256, p, p, p, p, p, None) == hb.HT_ERR_INVALID_ARG   # lengths must stay below 256

    # ht_verify_greedy_compact(logits, dtype, tokens, parent, root_pred, B, N, T, V, max_path, rows, pred, accept_len, accept_path,
    #                          next_token, status, k_cache, v_cache, desc, kv_len, new_kv_len, compact_status, stream)
    c = hb.CacheDesc(2, 1, 4, 64, 128, hb.HT_BF16, 4, 0, 0, 0)
    fused = lambda rows, desc, new_len: lib.ht_verify_greedy_compact(p, hb.HT_F16, p, p, None, 1, 4, 3, 100, 8, rows, p, p + 64, p, p, p,
                                                                     p, p, ctypes.byref(desc), p + 128, new_len, p, None)
    assert fused(2, c, p + 192) == hb.HT_ERR_INVALID_ARG          # rows < T
    assert fused(5, c, p + 192) == hb.HT_ERR_INVALID_ARG          # rows > N
    assert fused(0, c, p + 128) == hb.HT_ERR_INVALID_ARG          # new_kv_len is kv_len
    assert fused(0, c, p + 64) == hb.HT_ERR_INVALID_ARG           # new_kv_len is accept_len
    assert fused(0, hb.CacheDesc(2, 1, 4, 64, 128, hb.HT_BF16, 5, 0, 0, 0), p + 192) == hb.HT_ERR_INVALID_ARG    # the descriptor's N is not the logits'
    assert fused(0, hb.CacheDesc(2, 0, 4, 64, 128, hb.HT_BF16, 4, 0, 0, 0), p + 192) == hb.HT_ERR_INVALID_ARG    # nor its B

    c = hb.CacheDesc(2, 1, 4, 64, 128, hb.HT_BF16, 8, 0, 0, 0)
    assert lib.ht_kv_compact(p, p, ctypes.byref(c), p, p, p, 65, p, p, None) == hb.HT_ERR_INVALID_ARG
    assert lib.ht_kv_compact(None, p, ctypes.byref(c), p, p, p, 8, p, p, None) == hb.HT_ERR_INVALID_ARG
    assert lib.ht_kv_compact(p, p, ctypes.byref(c), p, p + 64, p + 128, 8, p, p + 192, None) == hb.HT_ERR_INVALID_ARG   # new_kv_len is kv_len
    assert b"overlap" in lib.ht_last_error_string()
    assert lib.ht_kv_compact(p, p, ctypes.byref(c), p, p + 64, p + 128, 8, p + 64, p + 192, None) == hb.HT_ERR_INVALID_ARG   # ... is accept_len
    c = hb.CacheDesc(2, 1, 4, 64, 3, hb.HT_BF16, 8, 0, 0, 0)                   # 6-byte rows
    assert lib.ht_kv_compact(p, p, ctypes.byref(c), p, p, p, 8, p, p, None) == hb.HT_ERR_UNSUPPORTED

    d = hb.AttnDesc(1, 4, 4, 4, 128, 64, hb.HT_BF16, 0.0, 0, 0, 0, 0)
    lib.ht_rope_kv_append.argtypes = [ctypes.POINTER(hb.AttnDesc)] + [ctypes.c_void_p] * 5 + [ctypes.c_float] + [ctypes.c_void_p] * 5
    assert lib.ht_rope_kv_append(ctypes.byref(d), p, p, p, p, p, 1.0, p, p, p, p, None) == hb.HT_ERR_INVALID_ARG     # base must exceed 1
    assert lib.ht_rope_kv_append(ctypes.byref(d), p, p, None, p, p, 10000.0, p, p, p, p, None) == hb.HT_ERR_INVALID_ARG
    assert lib.ht_rope_kv_append(ctypes.byref(d), p, p + 4, p, p, p, 10000.0, p, p, p, p, None) == hb.HT_ERR_INVALID_ARG

    # ht_draft_tree(logits, dtype, B, rows, V, first_row, P, K, tmpl_parent, tmpl_rank, T, root, base, topk, tokens, pos, status, stream)
    assert lib.ht_draft_tree(p, hb.HT_F16, 1, 10, 100, 7, 3, 17, p, p, 5, None, p, p, p, p, p, None) == hb.HT_ERR_INVALID_ARG   # K > 16
    assert lib.ht_draft_tree(p, hb.HT_F16, 1, 10, 100, 8, 3, 4, p, p, 5, None, p, p, p, p, p, None) == hb.HT_ERR_INVALID_ARG    # rows 8..10 of 10
    assert lib.ht_draft_tree(p, hb.HT_F16, 1, 10, 3, 7, 3, 4, p, p, 5, None, p, p, p, p, p, None) == hb.HT_ERR_INVALID_ARG      # K > V
    assert lib.ht_draft_tree(p, hb.HT_F16, 1, 10, 100, 7, 3, 4, p, None, 5, None, p, p, p, p, p, None) == hb.HT_ERR_INVALID_ARG
    assert lib.ht_draft_tree(None, hb.HT_F16, 0, 10, 100, 7, 3, 4, None, None, 5, None, None, None, None, None, None, None) == hb.HT_OK


def test_binding_refuses_cpu_tensors_and_has_no_fallback():
    import torch
    from paper_2404_12022_b200 import binding as hb
    with pytest.raises(ValueError):
        hb.transfer(torch.zeros(1, 8), torch.zeros(1, 8, 8))
    src = open(os.path.join(ROOT, "paper_2404_12022_b200", "binding.py")).read()
    assert "oracle" not in src.replace("no fallback", "")


def _in_child(env, code):
    import subprocess
    import sys
    e = dict(os.environ)
    e.update(env)
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=e, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    return r.stdout, r.stderr


_KNOB_PROBE = """
import ctypes
from paper_2404_12022_b200 import binding as hb
lib = hb.load()
d = hb.AttnDesc(4, 91, 32, 32, 128, 4224, hb.HT_BF16, 0.0, 0, 0, 0, 0)
clean = hb.AttnDesc(4, 91, 32, 32, 128, 4224, hb.HT_BF16, 0.0, 0, 0, 0, hb.HT_ATTN_WORKSPACE_CLEAN)
print(lib.ht_tree_attention_launches(ctypes.byref(d)), lib.ht_tree_attention_launches(ctypes.byref(clean)),
      lib.ht_tree_attention_workspace(ctypes.byref(d)))
print(lib.ht_transfer(None, None, None, 0, 3, 8, hb.HT_F32, None))
"""


def test_knobs_of_the_environment(lib):
    """HT_FORCE_PATH, HT_SPLITS and HT_LOG are read by the library itself (once per process, so each setting gets a
    child process); the calls made here are answered on the host."""
    plain, err = _in_child({}, _KNOB_PROBE)
    assert plain.split()[:2] == ["2", "1"] and err.strip() == ""         # tensor-core kernel: with / without the counter kernel
    ws_plain = int(plain.split()[2])
    forced, _ = _in_child({"HT_FORCE_PATH": "simt"}, _KNOB_PROBE)
    assert forced.split()[0] == forced.split()[1] and forced.split()[0] in ("1", "2")   # the ALU kernel, whatever the flags
    assert int(forced.split()[2]) >= ws_plain                             # the workspace is the maximum over the kernels
    split, _ = _in_child({"HT_SPLITS": "4"}, _KNOB_PROBE)
    assert split.split()[:2] == ["2", "2"]                                 # split-KV ALU kernel + its merge
    out, err = _in_child({"HT_LOG": "1"}, _KNOB_PROBE)
    assert out.split()[3] == "0" and "[ht] ht_transfer B=0 k=3 d=8" in err
