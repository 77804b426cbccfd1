#!/usr/bin/env python
"""Benchmark of the Speculative-Streaming decode hot path on B200.

A step = one pass of the whole hot path over one batch of synthetic input: the attention of every
layer (plain tree-masked layers, then the N_s multi-stream layers), greedy tree verification and
KV compaction over all layers.  Default workload: the 7B-class shape the headline metric is quoted
on (32 layers, 32 heads x 128, L = 2048, 64-node tree, gamma = 4).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 7b] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is achieved HBM GB/s: the step's algorithmic bytes (each
input and output byte counted once) divided by the device time of the step, inputs resident in HBM.
For N > 1 every rank runs an independent replica on its own GPU (the path has no exchange step);
time is the max over ranks and value sums the bytes of all ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "msa_tree_attention_step_hbm_throughput"
UNIT = "GB/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="7b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--profile", action="store_true",
                    help="small run for ncu: W warm-up + K steps launched directly (no CUDA graph), "
                         "no component timings, no end-to-end leg, no CPU baseline")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy kernel)"
    return 6650.0, "fallback (earlier measurement on this pool)"


# ---- clocks --------------------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); smax.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower() == "active":
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---- oracle timing (CPU baseline / reference arm) -----------------------------------------------------
def oracle_sample(st, heads_per_layer: int = 2):
    """Times the oracle, as it stands, on a bounded sample of the workload: `heads_per_layer` heads of
    one plain and one MSA layer (sequence 0), the whole verification of sequence 0, and the compaction
    of sequence 0 over 4 layers.  Returns (bytes_processed, seconds, description, threads)."""
    import oracle
    c = st.cfg
    H, d, T, g = c.n_heads, c.head_dim, c.n_nodes, c.gamma
    L = int(st.kv_len[0])
    n_plain = c.n_layers - c.n_msa_layers
    layers = ([0] if n_plain > 0 else []) + [c.n_layers - 1]
    hp = min(heads_per_layer, H)
    inputs = [st.layer(l) for l in layers]
    lg = st.logits()
    s0, cap = int(st.kv_start[0]), int(st.kv_capacity[0])
    nbytes = 0
    t0 = time.perf_counter()
    layer_seconds = []
    for ly in inputs:
        gg = g if ly.is_msa else 0
        t_ly = time.perf_counter()
        oracle.msa_attention(st.parent[0], L, gg, st.sm_scale, ly.q_main[0], ly.k_cache[s0:s0 + cap],
                             ly.v_cache[s0:s0 + cap], None if gg == 0 else ly.q_spec[0],
                             None if gg == 0 else ly.k_spec[0], None if gg == 0 else ly.v_spec[0], heads=(0, hp))
        nbytes += (4 * L * d + 4 * T * d + 4 * T * gg * d + 4 * T * (1 + gg) * d) * hp
        layer_seconds.append((ly.is_msa, time.perf_counter() - t_ly))
    oracle_sample.layer_seconds = layer_seconds
    r = oracle.tree_verify(lg[0], st.draft_tokens[0], st.parent[0], path_cap=64)
    nbytes += 4 * T * c.vocab
    k4 = np.stack([inputs[-1].k_cache[s0:s0 + cap]] * 4)
    oracle.kv_compact(k4, k4, L, r["accept_len"], r["path"])
    nbytes += 2 * 2 * r["accept_len"] * H * d * 2 * 4
    dt = time.perf_counter() - t0
    desc = ("sequence 0: %d of %d heads of %d attention layer(s) (one plain, one multi-stream), full verification, "
            "compaction over 4 layers" % (hp, H, len(inputs)))
    return nbytes, dt, desc, oracle.max_threads()


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as fh:
            for ln in fh:
                if ln.startswith("model name"):
                    return ln.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def cpu_baseline(st):
    """The oracle, as it stands, on a bounded sample of the workload: once with every core the process may use
    and once with one thread.  The sampled heads are independent and equal in cost, so the time of a whole step
    (every head of every layer) is the sampled layers' time scaled by the head and layer counts."""
    import oracle
    c = st.cfg
    n_all = oracle.max_threads()
    b, t_all, desc, thr = oracle_sample(st)
    layer_secs = list(oracle_sample.layer_seconds)
    oracle.set_threads(1)
    try:
        _, t_one, _, _ = oracle_sample(st, heads_per_layer=1)
    finally:
        oracle.set_threads(n_all)
    # extrapolation of the all-core run: one plain and one multi-stream layer were timed on `hp` heads each
    hp = min(2, c.n_heads)
    scale_heads = c.n_heads / hp * c.batch
    n_plain = c.n_layers - c.n_msa_layers
    est_step_s = 0.0
    for is_msa, sec in layer_secs:                          # every head of every sequence of every layer of that kind
        est_step_s += sec * scale_heads * (c.n_msa_layers if is_msa else n_plain)
    return {"value": b / t_all / 1e9, "unit": UNIT, "cores": thr, "kind": "oracle", "sample": desc, "seconds": t_all,
            "one_thread": {"seconds": t_one, "sample_heads_per_layer": 1}, "cpu_model": cpu_model(),
            "cores_available": len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else None,
            "extrapolated_step_seconds": est_step_s,
            "extrapolation": "attention only: each sampled layer's time x (heads x sequences / sampled heads) x layers of its kind "
                             "(sequence 0's length stands for all sequences)"}


def run_reference(args):
    """Reference arm: the CPU oracle timed on host cores, on bounded samples of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2402_11131_b200 import workloads as W
    st = W.make_step(W.CONFIGS[args.workload])
    steps = max(1, min(args.steps, 5))
    warm = max(0, min(args.warmup, 1))
    for _ in range(warm):
        oracle_sample(st)
    tot_b, tot_t, desc, thr = 0, 0.0, "", 1
    for _ in range(steps):
        b, t, desc, thr = oracle_sample(st)
        tot_b += b; tot_t += t
    val = tot_b / tot_t / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warm, "ms_per_step": tot_t / steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "note": "CPU oracle on a bounded sample per step"},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": thr, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---- our arm -----------------------------------------------------------------------------------------
def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    from paper_2402_11131_b200 import api, build, replicas, workloads as W
    from paper_2402_11131_b200.step import DeviceStep
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    api.lib()

    names = list(W.CONFIGS) if args.workload == "all" else [args.workload]
    for workload in names:
        line = measure(args, workload, world, rank, local_rank)
        if line is not None:
            print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def measure(args, workload, world, rank, local_rank):
    """One workload: builds its device state, times the step and its components, returns the JSON line (rank 0)."""
    import torch
    import torch.distributed as dist
    from paper_2402_11131_b200 import api, replicas, workloads as W
    from paper_2402_11131_b200.step import DeviceStep
    cfg = W.CONFIGS[workload]
    st = W.make_step(cfg)
    if args.profile:
        run_profile(args, st)
        return None
    distinct = 2 if cfg.batch > 1 else None       # the ragged batch reuses two host-generated slabs
    dev = DeviceStep(st, distinct_slabs=distinct, pinned_host=not args.no_e2e)
    stream = torch.cuda.Stream()
    nl = len(dev.layers)

    # bytes of one step (each byte once)
    with torch.cuda.stream(stream):
        dev.run_verify(stream)
    stream.synchronize()
    acc = dev.accept_len.cpu().numpy()
    attn_bytes = sum(dev.attention_bytes(i) for i in range(nl))
    step_bytes = attn_bytes + dev.verify_bytes() + dev.compact_bytes(acc)
    attn_flops = sum(dev.attention_flops(i) for i in range(nl))

    # ---- capture the step, and the attention layers alone, into CUDA graphs -----------------------
    def capture(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            fn(stream)                           # warm (lazy kernel attributes are set outside capture)
            stream.synchronize()
            with torch.cuda.graph(g, stream=stream):
                n = fn(stream)
        return g, n

    g_step, launches_per_step = capture(dev.run_step)
    g_attn, _ = capture(dev.run_attention)
    plain_idx = [i for i in range(nl) if not dev.is_msa[i]]
    msa_idx = [i for i in range(nl) if dev.is_msa[i]]
    g_plain = capture(lambda s: dev.run_attention(s, only=plain_idx))[0] if plain_idx else None
    g_msa = capture(lambda s: dev.run_attention(s, only=msa_idx))[0] if msa_idx else None
    g_verify, _ = capture(dev.run_verify)
    g_compact, _ = capture(dev.run_compact)

    def time_graph(g, reps, warm):
        with torch.cuda.stream(stream):
            for _ in range(warm):
                g.replay()
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(reps):
                g.replay()
            e1.record(stream)
            stream.synchronize()
        return e0.elapsed_time(e1) / reps     # ms per replay

    # ---- the timed region ----------------------------------------------------------------------
    K, Wm = args.steps, max(args.warmup, 3)
    with torch.cuda.stream(stream):
        for _ in range(Wm):
            g_step.replay()
    stream.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(K):
            g_step.replay()
        e1.record(stream)
    stream.synchronize()
    torch.cuda.synchronize()
    step_ms = e0.elapsed_time(e1) / K
    # component timings (same graphs' kernels, timed alone) while the clock sampler still runs
    attn_ms = time_graph(g_attn, K, 3)
    plain_ms = time_graph(g_plain, K, 3) if g_plain else None
    msa_ms = time_graph(g_msa, K, 3) if g_msa else None
    verify_ms = time_graph(g_verify, K, 3)
    compact_ms = time_graph(g_compact, K, 3)
    clocks = sampler.stop() if rank == 0 else None
    if world > 1:
        step_ms = replicas.max_over_ranks(step_ms, "cuda")
        dist.barrier()
    status = api.ss_status(dev.attn_ws, stream) or api.ss_status(dev.verify_ws, stream)
    if status != 0:
        raise RuntimeError("device status %d after the timed region" % status)
    # workspace word 2: CTAs of unsplit row blocks that gave up their shared reference and ran their tiles twice
    started_over = int(dev.attn_ws.view(torch.int32)[2])

    # ---- the draft-management calls around the step (not part of it), each timed alone --------------
    draft_us = None
    if rank == 0:
        draft_us = time_draft_management(dev, stream, capture, time_graph, max(10, min(K, 100)))

    # ---- end to end: per-step inputs from pinned host memory, results read back ------------------
    e2e = None
    if not args.no_e2e:
        e2e = time_e2e(dev, stream, max(3, min(K, 50)), world)

    if rank != 0:
        return None

    peak, peak_src = measured_peaks()
    value = world * step_bytes / (step_ms * 1e-3) / 1e9
    attn_launch_us = attn_ms * 1e3 / nl
    achieved = (attn_bytes / nl) / (attn_launch_us * 1e-6) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload, "batch": cfg.batch, "n_layers": cfg.n_layers,
                   "n_msa_layers": cfg.n_msa_layers, "n_heads": cfg.n_heads, "head_dim": cfg.head_dim,
                   "prefix_len": [int(x) for x in st.kv_len] if cfg.batch > 1 else int(st.kv_len[0]),
                   "tree_nodes": cfg.n_nodes, "gamma": cfg.gamma, "vocab": cfg.vocab,
                   "parallelism": "replicas" if world > 1 else "single_gpu",
                   "l2": ("every layer streams its own KV slab; a step touches %.0f MB, more than twice the 126 MB L2"
                          if step_bytes > 2 * 126e6 else
                          "a step touches only %.1f MB and is not flushed from the 126 MB L2 between steps: "
                          "a parity-sized case, launch-bound, no bandwidth claim") % (step_bytes / 1e6),
                   "launch": "whole step replayed as one CUDA graph; attention launched with programmatic dependent launch",
                   "attention_flags": "SS_ATTN_PREFIX_STABLE (nothing in flight before an attention call writes a cached prefix)",
                   "component_timings": "us_plain_layer / us_msa_layer stream a different slab per launch (cold); us_verify / us_compact replay one kernel on L2-warm data"},
        "step_bytes": step_bytes, "pct_of_8TBs": value / world / 8000.0 * 100,
        "us_per_layer": attn_ms * 1e3 / nl,
        "us_plain_layer": None if plain_ms is None else plain_ms * 1e3 / len(plain_idx),
        "us_msa_layer": None if msa_ms is None else msa_ms * 1e3 / len(msa_idx),
        "us_verify": verify_ms * 1e3, "us_compact": compact_ms * 1e3,
        "draft_management_us": draft_us,
        "mean_accept_len": float(acc.mean()),
        "row_blocks_started_over": started_over,
        "attention_tflops": attn_flops / (attn_ms * 1e-3) / 1e12,
        "gpu_launches": launches_per_step * K,
        "clocks": clocks,
        "pct_of_measured_peak": value / world / peak * 100,
        "roofline": {"kernel": "msa_attention_small_kernel (plain layers) / msa_attention_kernel (multi-stream layers)", "bound": "hbm", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                     "bytes_per_launch": attn_bytes / nl, "us_per_launch": attn_launch_us,
                     "timed": "CUDA events around replays of a graph of the step's %d attention launches, right after the timed region" % nl,
                     "traffic": ncu_traffic() if workload == "7b" else None},
        "e2e": e2e,
    }
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(st)
    return line



def time_draft_management(dev, stream, capture, time_graph, reps):
    """Microseconds per call of the entry points that build, prune and otherwise verify a draft, at the
    workload's shapes (batch, tree size, streams, vocabulary, hidden = heads x head_dim), each replayed alone
    as a CUDA graph on L2-warm synthetic logits.  They run once per step at most; the step timed above does
    not contain them."""
    import torch
    from paper_2402_11131_b200 import api
    c = dev.cfg
    B, T, g, V = c.batch, c.n_nodes, max(1, c.gamma), c.vocab
    hidden = c.n_heads * c.head_dim
    gen = torch.Generator(device="cuda").manual_seed(1234)
    k = 4
    stream_logits = torch.randn((B, 1, g, V), device="cuda", generator=gen)
    node_logits = dev.logits if dev.logits.shape == (B, T, V) else torch.randn((B, T, V), device="cuda", generator=gen)
    uniforms = torch.rand((B, T), device="cuda", generator=gen)
    bonus = torch.zeros(B, dtype=torch.int32, device="cuda")
    new_tokens = torch.zeros((B, T), dtype=torch.int32, device="cuda")
    new_trees, pruned_trees = api.empty_trees(B), api.empty_trees(B)
    i32 = lambda *shape: torch.zeros(shape, dtype=torch.int32, device="cuda")
    f32 = lambda *shape: torch.zeros(shape, dtype=torch.float32, device="cuda")
    accept_len, accept_path, last_node, bonus_out, node_token = i32(B), i32(B, 64), i32(B), i32(B), i32(B, T)
    edge_prob, entropy, new_index, kept_nodes, kept_tokens = f32(B, T), f32(B, T), i32(B, T), i32(B, T), i32(B, T)
    ws_draft = api.workspace(api.ss_next_draft_workspace_bytes(B, g, V))
    ws_stats = api.workspace(api.ss_tree_prune_workspace_bytes(B, T, V))
    ws_sampled = api.workspace(api.ss_tree_verify_sampled_workspace_bytes(B, T, V))
    rows = B * T
    m_hidden = torch.randn((rows, hidden), device="cuda", generator=gen).to(torch.bfloat16)
    p_emb = torch.randn((g, hidden), device="cuda", generator=gen).to(torch.bfloat16)
    s_hidden = torch.empty((rows, g, hidden), dtype=torch.bfloat16, device="cuda")
    v_main = torch.randn((rows, hidden), device="cuda", generator=gen).to(torch.bfloat16)
    v_streams = torch.empty((rows, g, hidden), dtype=torch.bfloat16, device="cuda")
    calls = {
        "ss_next_draft": lambda s: api.ss_next_draft(stream_logits, None, bonus, k, T, new_tokens, new_trees, ws_draft, s),
        "ss_tree_prune": lambda s: api.ss_tree_prune(node_logits, dev.tokens, dev.trees, 0.01, edge_prob, new_index, kept_nodes,
                                                     kept_tokens, pruned_trees, ws_stats, s),
        "ss_tree_verify_soft": lambda s: api.ss_tree_verify_soft(node_logits, dev.tokens, dev.trees, 0.09, 0.3, accept_len, accept_path,
                                                                 last_node, bonus_out, edge_prob, entropy, ws_stats, s),
        "ss_tree_verify_sampled": lambda s: api.ss_tree_verify_sampled(node_logits, dev.tokens, dev.trees, uniforms, k, accept_len,
                                                                       accept_path, last_node, bonus_out, node_token, ws_sampled, s),
        "ss_stream_insert": lambda s: api.ss_stream_insert(m_hidden, p_emb, s_hidden, s),
        "ss_value_rotate": lambda s: api.ss_value_rotate(v_main, v_streams, 0.05, s),
    }
    out = {}
    for name, fn in calls.items():
        graph, _ = capture(fn)
        out[name] = time_graph(graph, reps, 3) * 1e3
    for ws in (ws_draft, ws_stats, ws_sampled):
        status = api.ss_status(ws, stream)
        if status != 0:
            raise RuntimeError("device status %d after the draft-management calls" % status)
    out["shapes"] = "batch %d, %d nodes, %d streams, vocabulary %d, top-%d, hidden %d" % (B, T, g, V, k, hidden)
    return out


def run_profile(args, st):
    """The step launched directly K times after W warm-up steps: the command ncu wraps."""
    import torch
    from paper_2402_11131_b200 import api
    from paper_2402_11131_b200.step import DeviceStep
    dev = DeviceStep(st, distinct_slabs=2 if st.cfg.batch > 1 else None)
    stream = torch.cuda.Stream()
    for _ in range(args.warmup):
        dev.run_step(stream)
    stream.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    n = 0
    for _ in range(args.steps):
        n += dev.run_step(stream)
    e1.record(stream)
    stream.synchronize()
    status = api.ss_status(dev.attn_ws, stream) or api.ss_status(dev.verify_ws, stream)
    print(json.dumps({"profile_run": True, "workload": args.workload, "steps": args.steps, "warmup": args.warmup,
                      "ms_per_step_direct_launch": e0.elapsed_time(e1) / max(1, args.steps), "gpu_launches": n,
                      "device_status": status}))


def ncu_traffic():
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, if present."""
    path = os.path.join(ROOT, "profiles", "msa_attention_7b_traffic.txt")
    if os.path.exists(path):
        with open(path) as fh:
            return json.load(fh).get("msa_attention_dram_bytes_per_launch")
    return None


def time_e2e(dev, stream, reps, world):
    """The same step driven through the public API with the step's inputs in pinned HOST memory:
    every step copies the queries, the stream K/V, the tree nodes' K/V, the logits, the draft tokens
    and the tree descriptors to the device, runs the C-ABI calls, and reads the verification result
    back.  The KV prefix is the cache, i.e. state left in HBM by earlier steps, not a step input."""
    import torch
    import torch.distributed as dist
    from paper_2402_11131_b200 import api
    st, c = dev.st, dev.cfg
    B, T = c.batch, c.n_nodes
    nl = len(dev.layers)
    # pinned host staging of the per-step inputs
    h_logits = dev.logits.cpu().pin_memory()
    h_tokens = dev.tokens.cpu().pin_memory()
    h_trees = dev.trees.cpu().pin_memory()
    h_tree_kv = []
    for b in range(B):
        lo = int(st.kv_start[b]) + int(st.kv_len[b])
        h_tree_kv.append((lo, dev.k_all[:, lo:lo + T].cpu().pin_memory(), dev.v_all[:, lo:lo + T].cpu().pin_memory()))
    h_out = {k: torch.empty_like(getattr(dev, k), device="cpu").pin_memory()
             for k in ("accept_len", "accept_path", "bonus_token", "last_node", "kv_len_out")}
    h2d = h_logits.numel() * 4 + h_tokens.numel() * 4 + h_trees.numel()
    for lo, hk, hv in h_tree_kv:
        h2d += 2 * hk.numel() * 2
    for h in dev.host_inputs:
        h2d += sum(t.numel() * 2 for t in h.values())
    d2h = sum(t.numel() * 4 for t in h_out.values())

    # Copies run on their own stream and the compute stream follows them layer by layer: a layer's attention is
    # launched once its queries (and stream K/V) have landed, so the step costs about what its copies cost.
    copy_stream = torch.cuda.Stream()
    Q_GROUP = 8
    ev_pre = torch.cuda.Event()
    ev_layer = [torch.cuda.Event() for _ in range(nl)]
    ev_tail = torch.cuda.Event()
    ev_done = torch.cuda.Event()

    def one_step():
        copy_stream.wait_event(ev_done)           # the previous step has read what is about to be overwritten
        with torch.cuda.stream(copy_stream):
            dev.trees.copy_(h_trees, non_blocking=True)
            for lo, hk, hv in h_tree_kv:
                dev.k_all[:, lo:lo + T].copy_(hk, non_blocking=True)
                dev.v_all[:, lo:lo + T].copy_(hv, non_blocking=True)
            ev_pre.record(copy_stream)
            for i, h in enumerate(dev.host_inputs):
                if i % Q_GROUP == 0:              # the main-stream queries of a few layers per copy
                    dev.q_main_all[i:i + Q_GROUP].copy_(dev.host_q_main_all[i:i + Q_GROUP], non_blocking=True)
                if "q_spec" in h:
                    dev.q_spec[i].copy_(h["q_spec"], non_blocking=True)
                    dev.k_spec[i].copy_(h["k_spec"], non_blocking=True)
                    dev.v_spec[i].copy_(h["v_spec"], non_blocking=True)
                ev_layer[i].record(copy_stream)
            dev.logits.copy_(h_logits, non_blocking=True)
            dev.tokens.copy_(h_tokens, non_blocking=True)
            ev_tail.record(copy_stream)
        with torch.cuda.stream(stream):
            stream.wait_event(ev_pre)
            for i in range(nl):
                stream.wait_event(ev_layer[i])
                dev.run_attention(stream, only=[i])
            stream.wait_event(ev_tail)
            dev.run_verify(stream)
            dev.run_compact(stream)
            for k, t in h_out.items():
                t.copy_(getattr(dev, k), non_blocking=True)
            ev_done.record(stream)
        stream.synchronize()

    ev_done.record(stream)
    for _ in range(3):
        one_step()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(reps):
        one_step()
    torch.cuda.synchronize()
    dt = (time.perf_counter() - t0) / reps
    if world > 1:
        from paper_2402_11131_b200 import replicas
        dt = replicas.max_over_ranks(dt, "cuda")
    acc = dev.accept_len.cpu().numpy()
    step_bytes = (sum(dev.attention_bytes(i) for i in range(nl)) + dev.verify_bytes() + dev.compact_bytes(acc))
    return {"value": world * step_bytes / dt / 1e9, "unit": UNIT, "ms_per_step": dt * 1e3,
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": reps,
            "note": "per-step inputs (queries, stream K/V, tree K/V, logits, tokens, trees) copied from pinned host "
                    "memory on a copy stream, each layer launched when its inputs have landed; the KV prefix is "
                    "resident cache state; results read back to the host"}


if __name__ == "__main__":
    main()
