"""Benchmark of the tree-verify step (one JSON line on stdout).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3|c1|c2|c4] [--impl reference]

A step is one pass of the whole hot path over one batch of synthetic input: per layer a
tree-attention call, the hidden-transfer projection at the transfer layer, greedy
verification of the logits and KV compaction over all layers.  Default workload: config 3
(LLaMA-7B-shaped full step: 32 layers, batch 4, KV length 4096, 88-node trees plus 3
pseudo positions, bf16), the largest single-GPU configuration that is a whole step.

The path does not shard (one GPU, no collectives): with --gpus N each rank runs an
independent replica ("replicas only") and the value is the sum over ranks divided by the
slowest rank's time.

--impl reference times the CPU oracle (plain fp64 C) on the host cores on a bounded sample
of the same workload; it is a deliberately slow baseline, not a target.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "tree_verify_step_hbm_gbs"
UNIT = "GB/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c3", choices=["c1", "c2", "c3", "c4"])
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--eager", action="store_true", help="enqueue every library call from the host instead of replaying a CUDA graph of the step")
    ap.add_argument("--no-extras", action="store_true", help="skip e2e, cpu baseline and per-kernel timing")
    ap.add_argument("--fused", action="store_true", help="verification and compaction as one launch (ht_verify_greedy_compact) instead of two calls")
    return ap.parse_args()


def make_workload(args):
    from paper_2404_12022_b200 import workloads as wl
    if args.workload == "c1":
        return wl.config_c1()
    if args.workload == "c2":
        return wl.config_c2()
    if args.workload == "c4":
        return wl.config_c4()
    return wl.config_c3()


def workload_config(w, n_gpus):
    return {"workload": w.name, "layers": w.layers, "batch": w.B, "q_heads": w.Hq, "kv_heads": w.Hkv,
            "head_dim": w.D, "kv_len": (w.kv_len[0] if len(set(w.kv_len)) == 1 else "ragged %d..%d" % (min(w.kv_len), max(w.kv_len))),
            "tree_nodes": w.T, "pseudo_rows": w.P, "hidden": w.d, "transfer_steps": w.k, "vocab": w.V,
            "parallelism": "replicas x%d" % n_gpus if n_gpus > 1 else "single GPU",
            "l2_policy": "inputs larger than L2 (KV cache of a step >> 126 MB)",
            "attention_flags": "HT_ATTN_WORKSPACE_CLEAN | HT_ATTN_CONTEXT_FINAL (the step keeps its workspace; lengths, trees "
                               "and context rows are final before a layer's call)"}


# ------------------------------------------------------------------------------------------
# CPU oracle sample (reference arm and cpu_baseline leg)
# ------------------------------------------------------------------------------------------

class OracleSample:
    """A bounded sample of the step for the CPU oracle: attention on a few (sequence, KV head)
    units of one post-transfer layer, the transfer projection, verification of all logits and
    compaction of one layer.  Inputs are the workload's own values, regenerated on the host."""

    def __init__(self, w, n_units=16):
        import dataclasses
        import numpy as np
        from oracle import ht_oracle
        from paper_2404_12022_b200 import workloads as wl
        self.np, self.oracle, self.w = np, ht_oracle, w
        ht_oracle.build()
        layer = w.layers - 1
        inp = wl.make_inputs(w, "cpu", layers=[layer])
        self.inp = inp
        f = lambda t: t.float().numpy()
        rng = np.random.default_rng(0)
        units = sorted({(int(rng.integers(w.B)), int(rng.integers(w.Hkv))) for _ in range(4 * n_units)})[:n_units]
        g = w.Hq // w.Hkv
        self.units = []
        for b, hk in units:
            L = w.kv_len[b]
            self.units.append((f(inp.q[0][b:b + 1, :, hk * g:(hk + 1) * g]), f(inp.k_cache[0, b:b + 1, hk:hk + 1, :L + w.N]),
                               f(inp.v_cache[0, b:b + 1, hk:hk + 1, :L + w.N]), np.array([L], np.int32),
                               inp.parent[b:b + 1].numpy()))
        self.h, self.W = f(inp.h_src), f(inp.W)
        self.logits = f(inp.logits)
        self.tokens, self.parent = inp.tokens.numpy(), inp.parent.numpy()
        self.root_pred = None if inp.root_pred is None else inp.root_pred.numpy()
        self.kview = inp.k_cache.view(torch_int_view(inp.k_cache)).numpy()
        self.vview = inp.v_cache.view(torch_int_view(inp.v_cache)).numpy()
        e = w.elem_bytes()
        attn_bytes = sum(2 * (int(u[3][0]) + w.N) * w.D * e + 2 * w.N * g * w.D * e for u in self.units)
        self.bytes = (attn_bytes + w.k * w.d * w.d * e + w.B * w.N * w.V * e +
                      4 * sum(inp.want_len) * w.Hkv * w.D * e)
        self.describe = ("attention on %d of %d (sequence, KV head) units of one layer, the transfer projection, "
                         "verification of all logits, compaction of one layer" % (len(self.units), w.B * w.Hkv))

    def run(self):
        o = self.oracle
        for q, k, v, L, par in self.units:
            o.tree_attention(q, k, v, L, par)
        o.transfer(self.h, self.W)
        pred, alen, apath, nxt, st = o.verify_greedy(self.logits, self.tokens, self.parent, self.root_pred,
                                                     self.w.max_path)
        o.kv_compact(self.kview, self.vview, self.w.N, self.np.array(self.w.kv_len, self.np.int32), alen, apath)


def torch_int_view(t):
    import torch
    return torch.int32 if t.dtype == torch.float32 else torch.int16


def time_oracle(sample, steps, warmup, budget_s=None):
    for _ in range(warmup):
        sample.run()
    t0 = time.perf_counter()
    done = 0
    for _ in range(steps):
        sample.run()
        done += 1
        if budget_s is not None and time.perf_counter() - t0 > budget_s:
            break
    dt = (time.perf_counter() - t0) / done
    return dt, done


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import ht_oracle
    w = make_workload(args)
    sample = OracleSample(w)
    dt, done = time_oracle(sample, args.steps, args.warmup)
    value = sample.bytes / dt / 1e9
    cores = ht_oracle.num_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": done, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, 1),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample.describe},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
# Native arm
# ------------------------------------------------------------------------------------------

class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        import torch
        self.proc = None
        try:
            uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", uuid, "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in out.strip().splitlines():
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# DRAM traffic per launch of the attention kernel on a c3 layer, from the ncu capture of the committed build summarised
# at the end of profiles/attn_tc_kernel_c3_layer.md (dram__bytes_read.sum + dram__bytes_write.sum, mean of two launches).  It is only
# reported while the kernel source is the one that was profiled.
NCU_TRAFFIC = {"workload": "c3_llama7b_step_bf16", "bytes_per_launch": 287.6e6,
               "source": ["paper_2404_12022_b200/csrc/attn_tc.cu", "paper_2404_12022_b200/csrc/attn_tc.cuh",
                          "paper_2404_12022_b200/csrc/ht_common.cuh"],
               "sha256": "eaae2896afb6cfc62190630292e100236acc25093f3c70e33ac50d261a13661e"}


def traffic_digest():
    """SHA-256 of the attention kernel's sources and of the compiler flags they are built with."""
    import hashlib
    from paper_2404_12022_b200 import build
    h = hashlib.sha256()
    for f in NCU_TRAFFIC["source"]:
        h.update(open(os.path.join(ROOT, f), "rb").read())
    h.update(" ".join(build.NVCC_FLAGS).encode())
    return h.hexdigest()


def ncu_traffic(w):
    try:
        digest = traffic_digest()
    except OSError:
        return None
    if digest != NCU_TRAFFIC["sha256"] or w.name != NCU_TRAFFIC["workload"] or w.kv_len[0] != 4096 or w.B != 4:
        return None
    return NCU_TRAFFIC["bytes_per_launch"]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def replica_aggregate(ms_total_local, steps, step_bytes, world, device):
    """Whole-job figures of N independent replicas (the path does not shard): the step time is the
    slowest rank's, the value is all ranks' bytes over that time.  Uses the default process group
    when world > 1 (NCCL in the benchmark, gloo in the CPU test)."""
    ms_total = ms_total_local
    if world > 1:
        import torch
        import torch.distributed as dist
        t = torch.tensor([ms_total_local], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_step = ms_total / steps
    return ms_step, world * step_bytes / (ms_step * 1e-3) / 1e9


def run_native(args):
    import torch
    import torch.distributed as dist
    from paper_2404_12022_b200 import binding as hb
    from paper_2404_12022_b200 import workloads as wl
    from paper_2404_12022_b200.step import VerifyStep

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    w = make_workload(args)
    inp = wl.make_inputs(w, "cuda")
    step = VerifyStep(inp, fused=args.fused)
    stream = torch.cuda.current_stream().cuda_stream

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    step.run(stream)                      # eager once: per-device set-up inside the library
    torch.cuda.synchronize()
    if not args.eager:
        step.capture()                    # the step as one CUDA graph: same kernels, no host work between them
    run_step = (lambda: step.run(stream)) if args.eager else step.replay
    for _ in range(max(args.warmup, 3)):
        run_step()
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    marks[0].record()
    for i in range(args.steps):
        run_step()
        marks[i + 1].record()          # a mark per step (median and minimum); the figure is first mark to last
    barrier()
    ms_total = marks[0].elapsed_time(marks[-1])
    per_step_us = [marks[i].elapsed_time(marks[i + 1]) * 1e3 for i in range(args.steps)]
    clocks = sampler.stop() if sampler else None
    step_bytes = step.step_bytes()
    ms_step, value = replica_aggregate(ms_total, args.steps, step_bytes, world, "cuda")

    # correctness of what was just timed: status words and the seeded accepted lengths
    assert int(step.attn_status.abs().sum()) == 0 and int(step.verify_status.abs().sum()) == 0
    assert step.accept_len.cpu().tolist() == inp.want_len, "accepted lengths differ from the seeded ones"

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": w.dtype, "data": "synthetic", "config": workload_config(w, world),
            "step_us": ms_step * 1e3, "step_us_median": statistics.median(per_step_us), "step_us_min": min(per_step_us),
            "step_bytes": step_bytes, "clocks": clocks,
            "launch": "eager C-ABI calls" if args.eager else "CUDA graph of the step's C-ABI calls"}
    # launches of this library's kernels per step: the attention calls' (ht_tree_attention_launches), transfer (one
    # per batch slice of 16), verification with the compaction in the same launch
    line["gpu_launches"] = args.steps * (sum(kernels_per_attention(step, i) for i in range(step.layers)) + ((w.B + 15) // 16) + (1 if step.fused else 2))    # + transfer, verification and compaction (one kernel when fused)

    if rank == 0 and not args.no_extras:
        line["roofline"], line["kernels"] = per_kernel_pass(args, step, stream, torch)
        line["sustained"] = sustained_pass(run_step, step, local, line["kernels"]["attention"]["share"], torch)
        line["e2e"] = e2e_pass(args, step, inp, torch, world)
        sample = OracleSample(w)
        dt, done = time_oracle(sample, 1000, 0, budget_s=12.0)
        from oracle import ht_oracle
        line["cpu_baseline"] = {"value": sample.bytes / dt / 1e9, "unit": UNIT, "cores": ht_oracle.num_threads(),
                                "kind": "oracle", "sample": sample.describe + " (%d passes, %.2f s each)" % (done, dt)}
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)


def sustained_pass(run_step, step, device_index, attention_share, torch, seconds=2.0):
    """The same step replayed back to back for at least `seconds`, with the SM clock sampled meanwhile: what the
    step costs once the power cap has settled the clocks (the timed run above is a burst).  ms x MHz tells how much
    of a difference between two runs is clock."""
    peak, _ = measured_peaks()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    run_step()
    torch.cuda.synchronize()
    sampler = ClockSampler(device_index)
    t0 = time.perf_counter()
    n = 0
    e0.record()
    while time.perf_counter() - t0 < seconds:
        for _ in range(50):
            run_step()
        n += 50
        torch.cuda.synchronize()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / n
    attn_bytes = sum(step.attention_bytes(i) for i in range(step.layers))
    attn_gbs = attn_bytes / (ms * 1e-3 * attention_share) / 1e9
    return {"steps": n, "ms_per_step": ms, "value": step.step_bytes() / (ms * 1e-3) / 1e9, "unit": UNIT,
            "sm_mhz": clocks["sm_mhz"], "reasons": clocks["reasons"],
            "ms_x_mhz": ms * clocks["sm_mhz"] if clocks["sm_mhz"] else None,
            "attention_gbs": attn_gbs, "attention_frac": attn_gbs / peak,
            "note": "attention_gbs = attention bytes of a step / (the step's sustained time x the attention calls' share of the per-kernel pass)"}


def kernels_per_attention(step, i):
    """Kernels layer i's attention call enqueues (the attention kernel, and with it the one that zeroes its tickets)."""
    from paper_2404_12022_b200 import binding as hb
    return hb.tree_attention_launches(step.descs[i])


def per_kernel_pass(args, step, stream, torch):
    """Same steps again with CUDA events on the launching stream: one pair around every run of
    consecutive attention calls (an event between two launches would add its own gap to each of them, and
    would break the chain in which a call is set up while the one before it finishes), one pair around
    each of the other calls."""
    n = min(args.steps, 10)
    names = ["attention", "transfer"] + (["verify_compact"] if step.fused else ["verify", "compact"])
    ev = {k: [] for k in names}

    def pair():
        return torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(name, fn):
        a, b = pair(); a.record(); fn(); b.record(); ev[name].append((a, b))

    # In the launch mode of the timed steps: a run of attention calls is replayed from a CUDA graph of its own (or,
    # with --eager, enqueued call by call).
    run_graphs = {}

    def attention_run(lo, hi):
        if hi <= lo:
            return
        if not args.eager and (lo, hi) not in run_graphs:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side), torch.cuda.graph(g, stream=side):
                for i in range(lo, hi):
                    step.attention(i, side.cuda_stream)
            torch.cuda.current_stream().wait_stream(side)
            run_graphs[(lo, hi)] = g
        a, b = pair(); a.record()
        if args.eager:
            for i in range(lo, hi):
                step.attention(i, stream)
        else:
            run_graphs[(lo, hi)].replay()
        b.record(); ev["attention"].append((a, b, list(range(lo, hi))))

    cut = min(step.transfer_at, step.layers)
    for _ in range(n):
        attention_run(0, cut)
        timed("transfer", lambda: step.transfer(stream))
        attention_run(cut, step.layers)
        if step.fused:
            timed("verify_compact", lambda: step.verify_compact(stream))
        else:
            timed("verify", lambda: step.verify(stream))
            timed("compact", lambda: step.compact(stream))
    torch.cuda.synchronize()
    tot = {k: sum(x[0].elapsed_time(x[1]) for x in v) for k, v in ev.items()}
    all_ms = sum(tot.values())
    layers = [i for x in ev["attention"] for i in x[2]]
    attn_ms = tot["attention"] / len(layers)
    attn_bytes = sum(step.attention_bytes(i) for i in layers) / len(layers)
    attn_flops = sum(step.attention_flops(i) for i in layers) / len(layers)
    peak, how = measured_peaks()
    achieved = attn_bytes / (attn_ms * 1e-3) / 1e9
    roofline = {"kernel": "ht_tree_attention", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "frac_of_nominal_8tbs": achieved / 8000.0, "peak_source": how,
                "traffic": ncu_traffic(step.w), "bytes_per_launch": attn_bytes, "us_per_launch": attn_ms * 1e3,
                "tflops": attn_flops / (attn_ms * 1e-3) / 1e12}
    bytes_of = {"transfer": step.transfer_bytes(), "verify": step.verify_bytes(), "compact": step.compact_bytes(),
                "verify_compact": step.verify_bytes() + step.compact_bytes()}
    kernels = {"attention": {"us": attn_ms * 1e3, "share": tot["attention"] / all_ms, "gbs": achieved}}
    for k in names[1:]:
        us = tot[k] / len(ev[k]) * 1e3
        kernels[k] = {"us": us, "share": tot[k] / all_ms, "gbs": bytes_of[k] / (us * 1e-6) / 1e9}
    return roofline, kernels


def e2e_pass(args, step, inp, torch, world):
    """The same step with its per-step inputs arriving from pinned host memory and its results
    read back: q of every layer, the new K/V rows of the tree, logits, tree structure and the
    source hidden state go host -> device; attention outputs, pseudo hidden states and the
    acceptance results come back.  The KV cache and the transfer weights are resident state.
    The new rows reach the cache tail through ht_rope_kv_append (position 0 for every row: the
    rotation by angle 0 is exact, so the step computes on the same values as the device-resident
    runs)."""
    from paper_2404_12022_b200 import binding as hb
    w = step.w
    n = min(args.steps, 5)
    dev = inp.k_cache.device
    pin = lambda t: t.cpu().pin_memory()
    L = torch.tensor(w.kv_len, device=dev)
    idx = (L[:, None] + torch.arange(w.N, device=dev)[None]).long()          # [B, N] cache rows of the tree
    gather = lambda c: torch.stack([c[:, b][:, :, idx[b]] for b in range(w.B)], 1).permute(0, 1, 3, 2, 4).contiguous()
    all_k, all_v = gather(inp.k_cache), gather(inp.v_cache)                      # [layers, B, N, Hkv, D]
    rows_of = [q.shape[1] for q in inp.q]                                        # layers ahead of the transfer have no pseudo rows
    # One pinned buffer and one device buffer per layer hold q | k | v back to back, so a layer's inputs
    # travel as one copy.
    host_in, dev_in, host_q, host_k, host_v, dev_q, dev_k, dev_v = [], [], [], [], [], [], [], []
    for i, r in enumerate(rows_of):
        parts = [inp.q[i], all_k[i][:, :r].contiguous(), all_v[i][:, :r].contiguous()]
        total = sum(t.numel() for t in parts)
        hbuf = torch.empty(total, dtype=parts[0].dtype).pin_memory()
        dbuf = torch.empty(total, dtype=parts[0].dtype, device=dev)
        views_h, views_d, at = [], [], 0
        for t in parts:
            views_h.append(hbuf[at:at + t.numel()].view(t.shape))
            views_d.append(dbuf[at:at + t.numel()].view(t.shape))
            views_h[-1].copy_(t)
            at += t.numel()
        host_in.append(hbuf); dev_in.append(dbuf)
        host_q.append(views_h[0]); host_k.append(views_h[1]); host_v.append(views_h[2])
        dev_q.append(views_d[0]); dev_k.append(views_d[1]); dev_v.append(views_d[2])
    del all_k, all_v
    pos0 = [torch.zeros((w.B, r), dtype=torch.int32, device=dev) for r in rows_of]
    host_small = [pin(t) for t in (inp.logits, inp.parent, inp.parent_tree, inp.tokens, inp.h_src, inp.kv_len)]
    host_rp = pin(inp.root_pred) if inp.root_pred is not None else None
    small_targets = [inp.logits, inp.parent, inp.parent_tree, inp.tokens, inp.h_src, inp.kv_len]
    host_out = [torch.empty_like(o, device="cpu").pin_memory() for o in step.outs]
    host_res = [torch.empty_like(t, device="cpu").pin_memory() for t in
                (step.pseudo, step.pred, step.accept_len, step.accept_path, step.next_token, step.new_kv_len)]
    res_src = [step.pseudo, step.pred, step.accept_len, step.accept_path, step.next_token, step.new_kv_len]
    h2d = sum(t.numel() * t.element_size() for t in host_q + host_k + host_v + host_small + ([host_rp] if host_rp is not None else []))
    d2h = sum(t.numel() * t.element_size() for t in host_out + host_res)
    stream = torch.cuda.current_stream().cuda_stream

    copy_in, copy_out, place = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    comp = torch.cuda.current_stream()
    k_per_layer = len(host_k)
    ev_in = [torch.cuda.Event() for _ in range(step.layers)]
    ev_out = [torch.cuda.Event() for _ in range(step.layers)]
    ev_copied = [torch.cuda.Event() for _ in range(step.layers)]
    ev_small, ev_done = torch.cuda.Event(), torch.cuda.Event()
    assert k_per_layer == step.layers

    def one():
        """Layer i's inputs travel on a copy stream while layer i-1 computes; its output travels back
        on another while layer i+1 computes.  Everything a step reads arrives from the host inside
        the timed region, everything it produces is back on the host before the clock stops."""
        with torch.cuda.stream(copy_in):
            for t, h in zip(small_targets, host_small):
                t.copy_(h, non_blocking=True)
            if host_rp is not None:
                inp.root_pred.copy_(host_rp, non_blocking=True)
            ev_small.record(copy_in)
            for i in range(step.layers):
                dev_in[i].copy_(host_in[i], non_blocking=True)
                ev_copied[i].record(copy_in)
        with torch.cuda.stream(place):                     # the rows' placement runs beside the next layer's copies
            place.wait_event(ev_small)
            for i in range(step.layers):
                place.wait_event(ev_copied[i])
                hb.rope_kv_append(dev_q[i], dev_k[i], dev_v[i], pos0[i], inp.kv_len, inp.k_cache[i], inp.v_cache[i],
                                  q_out=inp.q[i])
                ev_in[i].record(place)
        comp.wait_event(ev_small)
        for i in range(step.layers):
            comp.wait_event(ev_in[i])
            if i == step.transfer_at:
                step.transfer(stream)
            step.attention(i, stream)
            ev_out[i].record(comp)
            with torch.cuda.stream(copy_out):
                copy_out.wait_event(ev_out[i])
                host_out[i].copy_(step.outs[i], non_blocking=True)
        if step.transfer_at >= step.layers:
            step.transfer(stream)
        if step.fused:
            step.verify_compact(stream)
        else:
            step.verify(stream)
            step.compact(stream)
        for s, h in zip(res_src, host_res):
            h.copy_(s, non_blocking=True)
        torch.cuda.synchronize()

    one()
    one()
    t0 = time.perf_counter()
    for _ in range(n):
        one()
    dt = (time.perf_counter() - t0) / n
    return {"value": world * step.step_bytes() / dt / 1e9, "unit": UNIT, "ms_per_step": dt * 1e3,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "note": "KV cache and transfer weights resident; per-step inputs from pinned host memory, copies of layer i+1 overlap the kernels of layer i"}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_native(args)


if __name__ == "__main__":
    main()
