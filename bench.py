"""Benchmark of the tree-verification step (n_layers x falcon_tree_attn +
falcon_tree_accept + falcon_kv_compact) on synthetic Vicuna/LLaMA2-shaped inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload v7b] [--impl falcon|reference]

Prints ONE JSON line.  `value` is whole-job verify steps/s with every input
resident in HBM (the step replayed as CUDA graphs, device-timed with CUDA
events); `e2e` is the same step driven from pinned host buffers with the
host<->device copies inside the timed region; `roofline` is the attention
kernel's algorithmic bytes per launch over its measured launch time;
`cpu_baseline` is the CPU oracle timed on a bounded sample of the same workload.
With --impl reference the oracle itself is the timed arm.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2412_12639_b200 import synth  # noqa: E402

METRIC = "tree-verify steps/sec"
UNIT = "steps/s"


# --------------------------------------------------------------------------- bytes
def attn_bytes_per_layer(spec, tb) -> int:
    """Algorithmic bytes of one attention launch: K and V rows of prefix+tree once, q read, out written."""
    total = 0
    for b in range(tb.batch):
        L, T = int(tb.prefix_len[b]), tb.tree_size(b)
        total += 2 * spec.n_kv_heads * (L + T) * spec.head_dim * 2 + 2 * T * spec.n_q_heads * spec.head_dim * 2 + 4 * T
    return total


def accept_bytes(spec, tb) -> int:
    return 4 * tb.total_nodes * spec.vocab + 12 * tb.total_nodes


def recorded_traffic(workload: str, kernel: str, stem: str = "tree_attn_%s"):
    """DRAM bytes per launch from the committed ncu summary of this workload and kernel (attention: "tc", "tck";
    stem "lm_head_argmax" for that kernel), or None when there is none or the kernel source has changed since
    the counters were taken."""
    import hashlib
    import re
    name = stem % kernel if "%s" in stem else stem
    try:
        text = open(os.path.join(ROOT, "profiles", "%s_%s_ncu.md" % (name, workload))).read()
        src = open(os.path.join(ROOT, "paper_2412_12639_b200", "csrc", "%s.cu" % name), "rb").read()
    except OSError:
        return None
    sha = re.search(r"kernel_source_sha256:\s*([0-9a-f]{64})", text)
    val = re.search(r"dram_bytes_per_launch:\s*(\d+)", text)
    if not sha or not val or sha.group(1) != hashlib.sha256(src).hexdigest():
        return None
    return int(val.group(1))


def traffic_note(workload: str, kernel: str):
    """The one-line remark a summary may carry next to its DRAM bytes (`traffic_note: ...`), or None."""
    import re
    try:
        text = open(os.path.join(ROOT, "profiles", "tree_attn_%s_%s_ncu.md" % (kernel, workload))).read()
    except OSError:
        return None
    m = re.search(r"traffic_note:\s*(.+)", text)
    return m.group(1).strip() if m else None


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for n, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------- oracle timing (CPU)
def time_oracle_step(spec, tb, logits, sample_layers: int, n_threads: int = 0):
    """Runs the CPU oracle on `sample_layers` layers of attention and compaction plus the full acceptance.
    With all layers this is one whole step; with fewer the per-layer time is extrapolated to the step.
    Returns (seconds per step, threads, description, extrapolated)."""
    import oracle
    scale = 1.0 / math.sqrt(spec.head_dim)
    t_attn = t_comp = 0.0
    g = oracle.argmax(logits, n_threads=n_threads)
    path, n_path, _ = oracle.tree_accept(tb.node_off, tb.parent, tb.token, g)
    for layer in range(sample_layers):
        q, k, v = synth.make_layer_qkv(spec, tb, layer)
        st = tuple(s // 2 for s in k.strides[:3])
        t0 = time.perf_counter()
        oracle.tree_attn(tb.node_off, tb.parent, tb.prefix_len, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, scale,
                         q, k, v, st, n_threads=n_threads)
        t1 = time.perf_counter()
        oracle.kv_compact(tb.node_off, tb.prefix_len, spec.n_kv_heads, spec.head_dim, k, st, k.shape[2], path, n_path)
        oracle.kv_compact(tb.node_off, tb.prefix_len, spec.n_kv_heads, spec.head_dim, v, st, v.shape[2], path, n_path)
        t2 = time.perf_counter()
        t_attn += t1 - t0
        t_comp += t2 - t1
    t0 = time.perf_counter()
    g = oracle.argmax(logits, n_threads=n_threads)
    oracle.tree_accept(tb.node_off, tb.parent, tb.token, g)
    t_acc = time.perf_counter() - t0
    step = (t_attn + t_comp) / sample_layers * spec.n_layers + t_acc
    extrapolated = sample_layers < spec.n_layers
    if extrapolated:
        desc = "%d of %d layers of attention+compaction and the full acceptance, extrapolated to one step" % (
            sample_layers, spec.n_layers)
    else:
        desc = "one whole step: all %d layers of attention+compaction and the acceptance" % spec.n_layers
    threads = n_threads if n_threads > 0 else oracle.max_threads()
    return step, threads, desc, extrapolated


def oracle_layer_flops(spec, tb) -> float:
    """Scalar double-precision flops of one layer of oracle attention."""
    return 4.0 * spec.head_dim * spec.n_q_heads * sum(
        tb.tree_size(b) * (int(tb.prefix_len[b]) + tb.tree_size(b)) for b in range(tb.batch))


def oracle_sample_layers(spec, tb, budget_flops: float = 40e9) -> int:
    """Layers of the oracle that fit a budget (about 40 GFLOP: roughly 10-30 s on a few cores); a whole step
    when it fits (the 7B-shaped step is 34 GFLOP)."""
    return max(1, min(spec.n_layers, int(budget_flops / max(oracle_layer_flops(spec, tb), 1.0))))


def config_of(args, spec, tb, world: int) -> dict:
    """The workload description both arms print, key for key."""
    step_bytes = spec.n_layers * attn_bytes_per_layer(spec, tb) + accept_bytes(spec, tb)
    return {"workload": args.workload, "batch": tb.batch, "n_layers": spec.n_layers, "n_q_heads": spec.n_q_heads,
            "n_kv_heads": spec.n_kv_heads, "head_dim": spec.head_dim, "prefix_len": tb.prefix_len.tolist(),
            "tree_nodes": np.diff(tb.node_off).tolist(), "vocab": spec.vocab,
            "parallelism": "replicas x%d (independent sequences, no collective)" % world,
            "l2": "inputs larger than L2: %.0f MB of distinct K/V, q and logits per step" % (step_bytes / 1e6),
            "timing": "CUDA graphs replayed on one stream, CUDA events, max over ranks"}


def run_reference(args):
    """The CPU oracle as the timed arm: whole steps whenever the run fits a few minutes, a stated sample of layers
    per step (and "extrapolated": true) otherwise."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = synth.SPECS[args.workload]
    tb = synth.make_trees(spec)
    logits = synth.make_logits(spec, tb)
    # one layer first, to know what a layer costs on this host; then as many layers per step as about 150 s allow
    t0 = time.perf_counter()
    time_oracle_step(spec, tb, logits, 1)
    per_layer = max(1e-4, (time.perf_counter() - t0))
    n_runs = max(1, args.steps + args.warmup)
    per_step_layers = max(1, min(spec.n_layers, int(150.0 / n_runs / per_layer)))
    for _ in range(args.warmup):
        time_oracle_step(spec, tb, logits, per_step_layers)
    times, threads, desc, extrapolated = [], 1, "", False
    for _ in range(args.steps):
        t, threads, desc, extrapolated = time_oracle_step(spec, tb, logits, per_step_layers)
        times.append(t)
    sec = sum(times) / len(times)
    val = 1.0 / sec
    cfg = config_of(args, spec, tb, 1)
    cfg["timing"] = "CPU oracle on the host cores, perf_counter"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": cfg, "extrapolated": extrapolated,
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def time_topm(ctx, binding, torch, dev, stream, logits_h, peak, m=20, copies=20, reps=20):
    """falcon_topm (m = 20, Appendix A) on the step's logits shape: `copies` distinct matrices (more than L2)
    in one CUDA graph, replayed; CUDA events on the launching stream.  Not part of the step."""
    N, V = logits_h.shape
    src = torch.from_numpy(logits_h).to(dev)
    mats = [src.clone() for _ in range(copies)]
    val = torch.empty((N, m), dtype=torch.float32, device=dev)
    idx = torch.empty((N, m), dtype=torch.int32, device=dev)
    calls = [binding.topm_args(N, V, x, V, m, val, idx) for x in mats]
    with torch.cuda.stream(stream):
        for a in calls:
            ctx.falcon_topm(a)              # the first call allocates scratch: before the capture
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for a in calls:
                ctx.falcon_topm(a)
        for _ in range(3):
            g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
        stream.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (reps * copies)
    nbytes = 4 * N * V + 8 * N * m
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"rows": N, "vocab": V, "m": m, "us_per_call": us, "bytes_per_call": nbytes,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                         "traffic": None}}


def time_sampled_accept(ctx, binding, torch, dev, stream, tree, tb, logits_h, peak, copies=20, reps=20):
    """falcon_tree_accept with temperature 1 (non-greedy decoding: every node's token drawn from its softmax with a
    caller-supplied uniform number) on the step's logits shape: `copies` distinct matrices (more than L2) in one
    CUDA graph, replayed; CUDA events on the launching stream.  Not part of the step."""
    N, V = logits_h.shape
    B = tb.batch
    src = torch.from_numpy(logits_h).to(dev)
    mats = [src.clone() for _ in range(copies)]
    g = torch.Generator(device=dev)
    g.manual_seed(13)
    u = torch.rand(N, device=dev, generator=g)
    tok = torch.empty(N, dtype=torch.int32, device=dev)
    path = torch.empty((B, 128), dtype=torch.int32, device=dev)
    n_path = torch.empty(B, dtype=torch.int32, device=dev)
    nxt = torch.empty(B, dtype=torch.int32, device=dev)
    calls = [binding.accept_args(tree, V, x, V, tok, path, 128, n_path, nxt, temperature=1.0, uniforms=u) for x in mats]
    with torch.cuda.stream(stream):
        for a in calls:
            ctx.falcon_tree_accept(a)       # the first call allocates scratch: before the capture
        stream.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=stream):
            for a in calls:
                ctx.falcon_tree_accept(a)
        for _ in range(3):
            gr.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            gr.replay()
        e1.record(stream)
        stream.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (reps * copies)
    nbytes = 4 * N * V + 4 * N
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"rows": N, "vocab": V, "temperature": 1.0, "us_per_call": us, "bytes_per_call": nbytes,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                         "traffic": None}}


def time_lm_head(ctx, binding, torch, dev, stream, n_rows, hidden, vocab, peak, workload, reps=10):
    """falcon_lm_head_argmax (Section 3.1, Eq. 6: the LM head applied to the nodes' features, greedy token only)
    at the workload's shape, hidden = query heads x head_dim: two distinct random heads alternate (together more
    than L2) in one CUDA graph, replayed; CUDA events on the launching stream.  Not part of the step."""
    g = torch.Generator(device=dev)
    g.manual_seed(11)
    heads = [torch.randn(vocab, hidden, device=dev, generator=g).bfloat16() for _ in range(2)]
    feat = torch.randn(n_rows, hidden, device=dev, generator=g).bfloat16()
    out = torch.zeros(n_rows, dtype=torch.int32, device=dev)
    calls = [binding.lm_argmax_args(n_rows, hidden, vocab, feat, hidden, w, hidden, out) for w in heads]
    per_graph = 4 * len(calls)
    with torch.cuda.stream(stream):
        for a in calls:
            ctx.falcon_lm_head_argmax(a)    # the first call sets the kernel's attributes: before the capture
        stream.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=stream):
            for _ in range(4):
                for a in calls:
                    ctx.falcon_lm_head_argmax(a)
        for _ in range(3):
            gr.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            gr.replay()
        e1.record(stream)
        stream.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (reps * per_graph)
    nbytes = 2 * vocab * hidden + 2 * n_rows * hidden + 4 * n_rows
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"rows": n_rows, "hidden": hidden, "vocab": vocab, "us_per_call": us, "bytes_per_call": nbytes,
            "useful_tflops": 2.0 * n_rows * hidden * vocab / (us * 1e-6) / 1e12,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                         "traffic": recorded_traffic(workload, "", stem="lm_head_argmax")}}


# --------------------------------------------------------------------------- GPU arm
ATTN_KERNELS = {"auto": 0, "simt": 1, "tc": 2, "tck": 3, "warp": 4}   # falcon.h FALCON_ATTN_*


def run_falcon(args):
    import torch
    import torch.distributed as dist
    import paper_2412_12639_b200 as falcon
    from paper_2412_12639_b200 import binding
    from paper_2412_12639_b200 import dist as fdist

    info = fdist.rank_info()
    world, rank, local = info.world, info.rank, info.local_rank
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    ctx = falcon.Context(local)

    spec = synth.SPECS[args.workload]
    # every rank verifies its own batch of sequences (independent problems: no exchange on this path)
    seed = fdist.shard_seed(spec.seed, rank)
    tb = synth.make_trees(spec, seed=seed)
    logits_h = synth.make_logits(spec, tb, seed=seed)
    s_cap = synth.cache_capacity(tb)
    B, N, Hq, Hkv, D, NL = tb.batch, tb.total_nodes, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.n_layers
    scale = 1.0 / math.sqrt(D)

    def i32(a):
        return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)

    # the tree arrays live in one device buffer (node_off, parent, token, prefix_len), which the end-to-end leg
    # refreshes from pinned host memory every step
    tree_host = torch.from_numpy(np.concatenate([tb.node_off, tb.parent, tb.token, tb.prefix_len]).astype(np.int32)
                                 ).pin_memory()
    tree_dev = tree_host.to(dev)
    o1, o2, o3 = B + 1, B + 1 + N, B + 1 + 2 * N
    node_off, parent, token, prefix = tree_dev[:o1], tree_dev[o1:o2], tree_dev[o2:o3], tree_dev[o3:]
    status = torch.zeros(B, dtype=torch.int32, device=dev)
    host_prefix = np.ascontiguousarray(tb.prefix_len, dtype=np.int32)   # the caller knows these: no device round trip
    host_node_off = np.ascontiguousarray(tb.node_off, dtype=np.int32)
    tree = binding.tree_desc(B, N, tb.max_tree, int(tb.prefix_len.max()), node_off, parent, prefix, token=token,
                             prefix_len_host=host_prefix, node_off_host=host_node_off, status=status)

    # all layers' caches in one allocation [NL, 2, B, Hkv, s_cap, D]; q and out [NL, N, Hq, D]
    cache = torch.empty((NL, 2, B, Hkv, s_cap, D), dtype=torch.bfloat16, device=dev)
    q_all = torch.empty((NL, N, Hq, D), dtype=torch.bfloat16, device=dev)
    out_all = torch.zeros_like(q_all)
    q_host = torch.empty((NL, N, Hq, D), dtype=torch.bfloat16).pin_memory()
    # the tree's own K/V rows of every layer, as the host hands them over each step (e2e leg)
    tree_rows = [(b, int(tb.prefix_len[b]), tb.tree_size(b)) for b in range(B)]
    tkv_host = [torch.empty((NL, 2, Hkv, T, D), dtype=torch.bfloat16).pin_memory() for (_, _, T) in tree_rows]
    for layer in range(NL):
        qh, kh, vh = synth.make_layer_qkv(spec, tb, layer, s_cap=s_cap, seed=seed)
        q_host[layer] = torch.from_numpy(qh.view(np.int16)).view(torch.bfloat16)
        kt = torch.from_numpy(kh.view(np.int16)).view(torch.bfloat16)
        vt = torch.from_numpy(vh.view(np.int16)).view(torch.bfloat16)
        cache[layer, 0].copy_(kt)
        cache[layer, 1].copy_(vt)
        for (b, L, T), th in zip(tree_rows, tkv_host):
            th[layer, 0] = kt[b, :, L:L + T]
            th[layer, 1] = vt[b, :, L:L + T]
    q_all.copy_(q_host)
    logits_host = torch.from_numpy(logits_h).pin_memory()
    logits = logits_host.to(dev)

    g = torch.zeros(N, dtype=torch.int32, device=dev)
    path = torch.zeros((B, 128), dtype=torch.int32, device=dev)
    n_path = torch.zeros(B, dtype=torch.int32, device=dev)
    nxt = torch.zeros(B, dtype=torch.int32, device=dev)
    new_len = torch.zeros(B, dtype=torch.int32, device=dev)
    result_dev = torch.zeros(3 * B + B * 128, dtype=torch.int32, device=dev)
    result_host = torch.zeros(3 * B + B * 128, dtype=torch.int32).pin_memory()
    kptr = torch.tensor([cache[l, 0].data_ptr() for l in range(NL)], dtype=torch.int64, device=dev)
    vptr = torch.tensor([cache[l, 1].data_ptr() for l in range(NL)], dtype=torch.int64, device=dev)
    strides = tuple(int(s) for s in cache[0, 0].stride()[:3])

    # The prefix rows were written in earlier steps: from the second layer on the kernel may ask for them while
    # the previous launch drains (the first layer follows the compaction of the previous step, which writes the
    # rows the new prefix ends with, so it makes no such promise), and each call names the next layer's caches,
    # whose prefix rows it may have brought into L2.
    attn = [binding.attn_args(tree, Hq, Hkv, D, scale, q_all[l], out_all[l], cache[l, 0], cache[l, 1], strides, s_cap,
                              flags=binding.ATTN_PREFIX_STABLE if l > 0 else 0, kernel=ATTN_KERNELS[args.attn_kernel],
                              next_k_cache=cache[l + 1, 0] if l + 1 < NL and not args.no_next_hint else None,
                              next_v_cache=cache[l + 1, 1] if l + 1 < NL and not args.no_next_hint else None)
            for l in range(NL)]
    acc = binding.accept_args(tree, spec.vocab, logits, logits.shape[1], g, path, 128, n_path, nxt)
    cmp_ = binding.compact_args(tree, NL, Hkv, D, kptr, vptr, strides, s_cap, path, 128, n_path, new_len)

    def launch_attn():
        for a in attn:
            ctx.falcon_tree_attn(a)

    def launch_tail():
        ctx.falcon_tree_accept(acc)
        ctx.falcon_kv_compact(cmp_)

    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        launch_attn()           # first calls allocate scratch: before any capture
        launch_tail()
        stream.synchronize()
        g_attn, g_tail = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_attn, stream=stream):
            launch_attn()
        with torch.cuda.graph(g_tail, stream=stream):
            launch_tail()

        def barrier():
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()

        # ---------------- device-resident steps ----------------
        for _ in range(args.warmup):
            g_attn.replay()
            g_tail.replay()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
        sampler = ClockSampler(local)
        barrier()
        sampler.start()
        t_wall = time.perf_counter()
        for s in range(args.steps):
            ev[s][0].record(stream)
            g_attn.replay()
            ev[s][1].record(stream)
            g_tail.replay()
            ev[s][2].record(stream)
        barrier()
        t_wall = time.perf_counter() - t_wall
        total_ms = ev[0][0].elapsed_time(ev[-1][2])
        attn_ms = sum(e[0].elapsed_time(e[1]) for e in ev)

        # ---------------- end to end from pinned host buffers ----------------
        def e2e_step():
            tree_dev.copy_(tree_host, non_blocking=True)
            q_all.copy_(q_host, non_blocking=True)
            for (b, L, T), th in zip(tree_rows, tkv_host):
                cache[:, :, b, :, L:L + T].copy_(th, non_blocking=True)
            logits.copy_(logits_host, non_blocking=True)
            g_attn.replay()
            g_tail.replay()
            result_dev[:B].copy_(n_path)
            result_dev[B:2 * B].copy_(nxt)
            result_dev[2 * B:3 * B].copy_(new_len)
            result_dev[3 * B:].copy_(path.view(-1))
            result_host.copy_(result_dev, non_blocking=True)
            stream.synchronize()

        for _ in range(max(1, min(args.warmup, 3))):
            e2e_step()
        e2e_steps = max(3, min(args.steps, 20))
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1)
        clocks = sampler.stop()

    total_ms, attn_ms, e2e_ms = fdist.max_over_ranks([total_ms, attn_ms, e2e_ms], dev)
    if not fdist.all_ok(not status.any().item(), dev):
        raise RuntimeError("device status words set on some rank (here: %s)" % status.tolist())

    h2d = (tree_host.numel() * 4 + q_host.numel() * 2 + sum(t.numel() for t in tkv_host) * 2 + logits_host.numel() * 4)
    d2h = result_host.numel() * 4
    ms_per_step = total_ms / args.steps
    per_launch_us = attn_ms / (args.steps * NL) * 1e3
    a_bytes = attn_bytes_per_layer(spec, tb)
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except OSError:
        pass
    peak = float(peaks.get("hbm_gbs", 6650.0))
    achieved = a_bytes / (per_launch_us * 1e-6) / 1e9
    kernel_name = {1: "simt", 2: "tc", 3: "tck", 4: "warp"}.get(ctx.falcon_tree_attn_kernel(attn[-1]), "?")
    traffic = recorded_traffic(args.workload, kernel_name)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---------------- outside the step: the selection that grows the tree (the row next to the hot path) ----
    topm = time_topm(ctx, binding, torch, dev, stream, logits_h, peak) if world == 1 else None
    sampled = time_sampled_accept(ctx, binding, torch, dev, stream, tree, tb, logits_h, peak) if world == 1 else None
    lm = (time_lm_head(ctx, binding, torch, dev, stream, tb.total_nodes, spec.n_q_heads * spec.head_dim, spec.vocab, peak,
                       args.workload) if world == 1 else None)

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        sl = oracle_sample_layers(spec, tb)
        sec, threads, desc, extrapolated = time_oracle_step(spec, tb, logits_h, sl)
        sec1, _, desc1, _ = time_oracle_step(spec, tb, logits_h, max(1, sl // 8), n_threads=1)
        cpu = {"value": 1.0 / sec, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc,
               "extrapolated": extrapolated,
               "single_thread": {"value": 1.0 / sec1, "unit": UNIT, "cores": 1, "sample": desc1}}

    line = {
        "metric": METRIC, "value": fdist.whole_job_rate(1.0, world, ms_per_step), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_of(args, spec, tb, world),
        "us_per_layer": per_launch_us,
        "roofline": {"bound": "hbm", "kernel": "falcon_tree_attn (tree_attn_%s.cu)" % kernel_name, "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic,
                     "traffic_note": traffic_note(args.workload, kernel_name) if traffic is not None else None,
                     "bytes_per_launch": a_bytes,
                     "us_per_launch": per_launch_us,
                     "peak_source": "MEASURED_PEAKS.json hbm_gbs" if peaks else "fallback 6650 GB/s"},
        "e2e": {"value": fdist.whole_job_rate(e2e_steps, world, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h},
        "gpu_launches": args.steps * (NL + 2),
        "clocks": clocks,
        "cpu_baseline": cpu,
        "extras": {"falcon_topm": topm, "falcon_lm_head_argmax": lm, "falcon_tree_accept_sampled": sampled},
        "wall_s_timed": t_wall,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="v7b", choices=sorted(synth.SPECS) + ["all"],
                    help="one of the five configurations (default: the metric's), or 'all': one JSON line each (1 GPU)")
    ap.add_argument("--impl", default="falcon", choices=["falcon", "reference"])
    ap.add_argument("--attn-kernel", default="auto", choices=sorted(ATTN_KERNELS),
                    help="which attention kernel falcon_tree_attn is asked for (auto = the library's choice)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-next-hint", action="store_true", help="do not name the next layer's caches to falcon_tree_attn")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "falcon":
        args.warmup = 3
    if args.workload == "all":
        # every configuration in a process of its own (each holds up to a few GB of caches), one line each
        for name in ("tiny", "v7b", "l13b", "l70b", "ragged"):
            cmd = [sys.executable, os.path.abspath(__file__), "--workload", name, "--steps", str(args.steps), "--warmup",
                   str(args.warmup), "--impl", args.impl, "--attn-kernel", args.attn_kernel, "--no-cpu-baseline"]
            if args.no_next_hint:
                cmd.append("--no-next-hint")
            r = subprocess.run(cmd, capture_output=True, text=True)
            sys.stdout.write(r.stdout)
            if r.returncode:
                sys.stderr.write(r.stderr[-2000:])
                sys.exit(r.returncode)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_falcon(args)


if __name__ == "__main__":
    main()
