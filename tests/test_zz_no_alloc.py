"""The allocation-free attention entry point against the ordinary one (collected last).

``ht_tree_attention_static`` serves callers that cannot hand the library a workspace
because they cannot allocate device memory at all; its split partials sit in an array
inside the library.  The test calls it through the C ABI twice in a row, on different
inputs, so that the second call runs on an array still holding the first call's partials,
and compares each result with what ``ht_tree_attention`` returns for the same inputs.
Both run the same kernel, so the results must agree to well within the parity tolerance
(1e-5 for fp32, 2e-3 + 1e-2 |ref| for bf16); each result is also held to the CPU oracle at
that tolerance.  The second call must leave the device's free memory as it found it, must
flag an illegal tree and a length that does not fit like the ordinary entry point does, and
sizes beyond the array must be refused.
"""
import numpy as np
import pytest
import torch

from paper_2404_12022_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _case(seed, dtype, B, N, Hq, Hkv, D, lens, cap):
    rng = np.random.default_rng(seed)
    q = wl.normal_tensor(seed, 1, (B, N, Hq, D), "cuda", 1.0, dtype)
    k = wl.normal_tensor(seed, 2, (B, Hkv, cap, D), "cuda", 1.0, dtype)
    v = wl.normal_tensor(seed, 3, (B, Hkv, cap, D), "cuda", 1.0, dtype)
    parent = np.full((B, N), -1, np.int32)
    for b in range(B):
        for r in range(1, N):
            parent[b, r] = rng.integers(-1, r)
    return q, k, v, torch.tensor(lens, dtype=torch.int32, device="cuda"), torch.from_numpy(parent).cuda()


def test_static_scratch_entry_point_matches_the_workspace_one_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2404_12022_b200 import binding as hb
    from oracle import ht_oracle
    ht_oracle.build()
    cases = [(101, torch.float32, 2, 37, 4, 2, 64, [513, 64], 640, 4),
             (102, torch.bfloat16, 1, 91, 8, 8, 128, [1000], 1152, 3)]
    for i, (seed, dtype, B, N, Hq, Hkv, D, lens, cap, splits) in enumerate(cases):
        q, k, v, kv_len, parent = _case(seed, dtype, B, N, Hq, Hkv, D, lens, cap)
        ref, st_ref = hb.tree_attention(q, k, v, kv_len, parent, num_splits=splits,
                                        flags=hb.HT_ATTN_FORCE_SIMT)
        out = torch.empty_like(q)
        status = torch.full((B,), -1, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        hb.tree_attention_static(q, k, v, kv_len, parent, out=out, status=status, num_splits=splits)
        torch.cuda.synchronize()
        if i > 0:                       # the first call may load the kernels' code; the second allocates nothing
            assert torch.cuda.mem_get_info()[0] == free_before
        assert status.cpu().tolist() == st_ref.cpu().tolist() == [0] * B
        want = ht_oracle.tree_attention(q.float().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy(),
                                        kv_len.cpu().numpy(), parent.cpu().numpy())
        for other in (ref.float().cpu().numpy().astype(np.float64), want):
            err = np.abs(out.float().cpu().numpy() - other)
            if dtype == torch.float32:
                assert float(err.max()) <= 1e-5
            else:
                assert bool((err <= 2e-3 + 1e-2 * np.abs(other)).all())
    # sequences only the device can find fault with are skipped and flagged, their rows left alone
    q, k, v, kv_len, parent = _case(104, torch.float32, 3, 9, 4, 2, 64, [10, 20, 30], 64)
    parent[1, 4] = 4
    kv_len[2] = 60
    out = torch.full_like(q, 7.0)
    out, status = hb.tree_attention_static(q, k, v, kv_len, parent, out=out, num_splits=2)
    ref, st_ref = hb.tree_attention(q, k, v, kv_len, parent, out=torch.full_like(q, 7.0), num_splits=2, flags=hb.HT_ATTN_FORCE_SIMT)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == st_ref.cpu().tolist() == [hb.HT_STATUS_OK, hb.HT_STATUS_BAD_TREE, hb.HT_STATUS_BAD_LEN]
    assert bool((out[1:] == 7.0).all()) and float((out[0] - ref[0]).abs().max()) <= 1e-5
    # a problem whose partials do not fit in the built-in array is refused, not truncated
    q, k, v, kv_len, parent = _case(103, torch.float32, 4, 200, 16, 16, 128, [300] * 4, 512)
    with pytest.raises(hb.HtError) as e:
        hb.tree_attention_static(q, k, v, kv_len, parent, num_splits=8)
    assert e.value.code == hb.HT_ERR_WORKSPACE and "built-in scratch" in str(e.value)
    # ... while the same problem without splits needs no scratch at all
    out, status = hb.tree_attention_static(q, k, v, kv_len, parent, num_splits=1)
    ref, _ = hb.tree_attention(q, k, v, kv_len, parent, num_splits=1, flags=hb.HT_ATTN_FORCE_SIMT)
    torch.cuda.synchronize()
    assert float((out - ref).abs().max()) <= 1e-5
