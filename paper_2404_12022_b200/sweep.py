"""Timing sweeps of single entry points, one JSON line per point (the results tables are made from these).

  python -m paper_2404_12022_b200.sweep attention --set configs|c5|c5-quick [--paged P] [--only TEXT] [--reps R]
  python -m paper_2404_12022_b200.sweep transfer [--only TEXT] [--reps R]
  python -m paper_2404_12022_b200.sweep step --layers L [--kv KV] [--steps K]      (a small step, for profiler captures)
  python -m paper_2404_12022_b200.sweep peak                                        (copy and read-only streaming rates)

Protocol of the attention and transfer sweeps: CUDA events around a CUDA graph of at least 16 calls that rotate over
enough copies of the cache (of W) to exceed twice the L2, median of 5 replays.  This is not the step benchmark
(``bench.py`` at the repository root).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), float(p.get("bf16_tflops", 0.0)) or None
    return 6650.0, 1590.0


def sweep_points(which):
    import dataclasses
    from . import workloads as wl
    if which == "configs":
        c2 = wl.config_c2()
        return [c2, dataclasses.replace(c2, name="c2_at_kv2048", kv_len=[2048]), wl.config_c3(layers=1), wl.config_c4()]
    pts = wl.c5_points()
    if which == "c5-quick":
        pts = [p for p in pts if p[2] == 4 and p[1] in (16, 64, 256)]
    return [wl.config_c5(*p) for p in pts]


def run_attention(args):
    """CUDA-event time of ht_tree_attention per call, replayed from a CUDA graph of `reps` calls
    that rotate over enough copies of the cache to exceed twice the L2 (cold-L2 protocol)."""
    import torch
    from . import binding as hb
    from . import workloads as wl
    torch.cuda.set_device(0)
    peak, _ = measured_peaks()
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    for w in [x for x in sweep_points(args.set) if args.only in x.name]:
        inp = wl.make_inputs(w, "cuda", with_logits=False, with_transfer=False, layers=[w.layers - 1])
        q, kv_len, parent = inp.q[0], inp.kv_len, inp.parent
        e = w.elem_bytes()
        cache_bytes = 2 * inp.k_cache[0].numel() * e
        nbuf = int(min(64, max(2, -(-2 * l2 // cache_bytes))))
        ks = [inp.k_cache[0]] + [wl.normal_tensor(w.seed, 10 + i, tuple(inp.k_cache[0].shape), "cuda", 1.0, w.torch_dtype())
                                 for i in range(nbuf - 1)]
        vs = [inp.v_cache[0]] + [wl.normal_tensor(w.seed, 100 + i, tuple(inp.k_cache[0].shape), "cuda", 1.0, w.torch_dtype())
                                 for i in range(nbuf - 1)]
        out = torch.empty_like(q)
        st = torch.zeros(w.B, dtype=torch.int32, device="cuda")
        desc = hb.make_attn_desc(q, ks[0])
        ws = torch.zeros(max(hb.tree_attention_workspace(desc), 16), dtype=torch.uint8, device="cuda")
        # the workspace is zeroed once and left clean by every call, lengths, trees and caches are final: what a
        # decoding loop can promise
        clean = hb.HT_ATTN_WORKSPACE_CLEAN | hb.HT_ATTN_CONTEXT_FINAL
        reps = args.reps or max(nbuf, 16)
        call = lambda i: hb.tree_attention(q, ks[i % nbuf], vs[i % nbuf], kv_len, parent, out=out, workspace=ws, status=st,
                                           flags=clean)
        if args.paged:
            ps = args.paged
            B, Hkv, cap, D = ks[0].shape
            per = cap // ps
            assert per * ps == cap, "--paged must divide the cache capacity %d" % cap
            g = torch.Generator(device="cpu").manual_seed(w.seed)
            table = torch.randperm(B * per, generator=g).to(torch.int32).reshape(B, per).cuda()

            def to_pool(c):      # page table[b][i] of the pool holds rows [i ps, (i + 1) ps) of sequence b
                pool = torch.empty((B * per, Hkv, ps, D), dtype=c.dtype, device="cuda")
                pool[table.reshape(-1).long()] = c.view(B, Hkv, per, ps, D).permute(0, 2, 1, 3, 4).reshape(B * per, Hkv, ps, D)
                return pool
            ks = [to_pool(c) for c in ks]
            vs = [to_pool(c) for c in vs]
            call = lambda i: hb.tree_attention_paged(q, ks[i % nbuf], vs[i % nbuf], table, kv_len, parent, out=out,
                                                     workspace=ws, status=st, flags=hb.HT_ATTN_CONTEXT_FINAL)
        for i in range(3):
            call(i)
        torch.cuda.synchronize()
        graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side), torch.cuda.graph(graph, stream=side):
            for i in range(reps):
                call(i)
        torch.cuda.synchronize()
        graph.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        times = []
        for _ in range(5):
            e0.record(); graph.replay(); e1.record(); torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1) / reps * 1e3)
        us = statistics.median(times)
        rows = q.shape[1]
        byts = sum(2 * w.Hkv * (L + rows) * w.D * e for L in w.kv_len) + 2 * w.B * rows * w.Hq * w.D * e + 4 * w.B * rows
        flops = sum(4 * rows * w.Hq * (L + rows) * w.D for L in w.kv_len)
        assert int(st.abs().sum()) == 0
        print(json.dumps({"workload": w.name, "batch": w.B, "kv_len": w.kv_len[0] if len(set(w.kv_len)) == 1 else "ragged",
                          "rows": rows, "q_heads": w.Hq, "kv_heads": w.Hkv, "dtype": w.dtype, "us": round(us, 2),
                          "hbm_gbs": round(byts / us / 1e3, 1), "frac_of_measured_hbm": round(byts / us / 1e3 / peak, 3),
                          "frac_of_8tbs": round(byts / us / 1e3 / 8000.0, 3), "tflops": round(flops / us / 1e6, 1),
                          "flop_per_byte": round(flops / byts, 1), "cold_l2_copies": nbuf,
                          "cache": ("pages of %d rows" % args.paged) if args.paged else "contiguous"}), flush=True)
        del ks, vs, inp, ws, graph


# (name, source rows, k, d): the configurations' projections with pseudo states hanging off one node per
# sequence (B rows) and off every tree node (B x T rows)
TRANSFER_POINTS = [("c2_per_sequence", 1, 3, 4096), ("c3_per_sequence", 4, 3, 4096), ("c4_per_sequence", 8, 4, 5120),
                   ("c5_per_sequence_b16", 16, 3, 8192), ("c2_per_node", 88, 3, 4096), ("c3_per_node", 352, 3, 4096),
                   ("c4_per_node", 512, 4, 5120), ("c5_per_node_b4_t256", 1024, 3, 8192),
                   ("c5_per_node_b16_t256", 4096, 3, 8192)]


def run_transfer(args):
    """CUDA-event time of ht_transfer per call, replayed from a CUDA graph whose calls rotate over
    enough copies of W to exceed twice the L2."""
    import torch
    from . import binding as hb
    from . import workloads as wl
    torch.cuda.set_device(0)
    peak, tensor_peak = measured_peaks()
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    for name, B, k, d in [x for x in TRANSFER_POINTS if args.only in x[0]]:
        wbytes = k * d * d * 2
        ncopy = int(max(2, -(-2 * l2 // wbytes)))
        h = wl.normal_tensor(31, 1, (B, d), "cuda", 1.0, torch.bfloat16)
        Ws = [wl.normal_tensor(31, 2 + i, (k, d, d), "cuda", 0.02, torch.bfloat16) for i in range(ncopy)]
        out = torch.empty((B, k, d), dtype=torch.bfloat16, device="cuda")
        for i in range(3):
            hb.transfer(h, Ws[i % ncopy], out)
        torch.cuda.synchronize()
        reps = args.reps or ncopy * (4 if B <= 512 else 1)
        graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side), torch.cuda.graph(graph, stream=side):
            for i in range(reps):
                hb.transfer(h, Ws[i % ncopy], out)
        torch.cuda.synchronize()
        graph.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        times = []
        for _ in range(5):
            e0.record(); graph.replay(); e1.record(); torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1) / reps * 1e3)
        us = statistics.median(times)
        byts = wbytes + B * d * 2 + B * k * d * 2
        flops = 2.0 * B * k * d * d
        line = {"workload": "transfer_" + name, "rows": B, "k": k, "d": d, "dtype": "bf16", "us": round(us, 2),
                "hbm_gbs": round(byts / us / 1e3, 1), "frac_of_measured_hbm": round(byts / us / 1e3 / peak, 3),
                "tflops": round(flops / us / 1e6, 1), "flop_per_byte": round(flops / byts, 1), "cold_l2_copies": ncopy}
        if tensor_peak:
            line["frac_of_measured_bf16"] = round(flops / us / 1e6 / tensor_peak, 3)
        print(json.dumps(line), flush=True)
        del Ws, graph




def run_step(args):
    """A small step of config 3 (few layers, optionally a shorter cache), enqueued call by call: every launch is
    full-size per layer, so a profiler capture of a few launches stays small."""
    import torch
    from . import workloads as wl
    from .step import VerifyStep
    torch.cuda.set_device(0)
    w = wl.config_c3(layers=args.layers, kv=args.kv)
    inp = wl.make_inputs(w, "cuda")
    step = VerifyStep(inp, fused=args.fused)
    stream = torch.cuda.current_stream().cuda_stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        step.run(stream)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        step.run(stream)
    e1.record()
    torch.cuda.synchronize()
    assert int(step.attn_status.abs().sum()) == 0 and step.accept_len.cpu().tolist() == inp.want_len
    print(json.dumps({"workload": w.name, "layers": w.layers, "kv_len": w.kv_len[0], "steps": args.steps,
                      "ms_per_step": e0.elapsed_time(e1) / args.steps, "launch": "eager C-ABI calls"}), flush=True)


def run_peak(args):
    """Streaming rates of the device as plain library kernels reach them: a copy (read + write, what the measured
    peak file holds) and a read-only pass (the fastest of a few reductions), over 2 GiB, best of 10 with CUDA events."""
    import torch
    torch.cuda.set_device(0)
    n = 1 << 30
    a = torch.ones(n, dtype=torch.bfloat16, device="cuda")
    b = torch.empty_like(a)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def best(fn):
        ts = []
        for _ in range(10):
            e0.record(); fn(); e1.record(); torch.cuda.synchronize(); ts.append(e0.elapsed_time(e1))
        return min(ts)
    copy_ms = best(lambda: b.copy_(a))
    f32 = a.view(torch.float32)
    reads = {"sum_f32": lambda: torch.sum(f32), "max_f32": lambda: torch.max(f32), "sum_bf16": lambda: torch.sum(a),
             "count_nonzero_i32": lambda: torch.count_nonzero(a.view(torch.int32))}
    read_gbs = {k: round(n * 2 / best(fn) / 1e6, 1) for k, fn in reads.items()}
    print(json.dumps({"copy_gbs": round(2 * n * 2 / copy_ms / 1e6, 1), "read_only_gbs": max(read_gbs.values()), "read_only_by_op": read_gbs,
                      "bytes": n * 2, "how": "torch copy_ / the fastest of a few torch reductions over 2 GiB, best of 10 each"}), flush=True)


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    sub = ap.add_subparsers(dest="what", required=True)
    a = sub.add_parser("attention")
    a.add_argument("--set", default="configs", choices=["configs", "c5", "c5-quick"])
    a.add_argument("--paged", type=int, default=0, help="the cache cut into pages of this many rows, placed in a seeded random "
                   "order in a pool (ht_tree_attention_paged)")
    a.add_argument("--only", default="", help="keep the workloads whose name contains this text")
    a.add_argument("--reps", type=int, default=0, help="calls per graph (small captures)")
    t = sub.add_parser("transfer")
    t.add_argument("--only", default="")
    t.add_argument("--reps", type=int, default=0)
    s = sub.add_parser("step")
    s.add_argument("--layers", type=int, default=2)
    s.add_argument("--kv", type=int, default=4096)
    s.add_argument("--steps", type=int, default=1)
    s.add_argument("--fused", action="store_true")
    sub.add_parser("peak")
    args = ap.parse_args()
    {"attention": run_attention, "transfer": run_transfer, "step": run_step, "peak": run_peak}[args.what](args)


if __name__ == "__main__":
    main()
