#!/usr/bin/env python
"""Benchmark of the DDTree verify round (build + layers x tree attention + accept) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--variant lit|peak]
    python bench.py --impl reference ...      # times the CPU oracle on a bounded sample

One step = one decoding round of the chosen workload: ddtree_build on the drafter logits, one
ddtree_tree_attention call per layer (distinct K/V cache per layer, tree mask taken on the device
from the build of the same step) and ddtree_accept on the target logits.  With N > 1 (torchrun)
every rank runs an independent replica of the workload (requests are independent; there is no
data-path collective), so scaling is "weak" and the value is the sum over ranks.

Prints one JSON line (rank 0).
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_12989_b200 import workloads as wl  # noqa: E402

METRIC = "ddtree_verify_rounds_per_s"
UNIT = "rounds/s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of tree_attention_bf16_kernel on the
# workload, from the ncu captures summarised in profiles/tree_attention_bf16_config{1,2}.txt.
NCU_TRAFFIC_BYTES = {1: 17653504, 2: 74303232}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], tflops=p["bf16_tflops_sustained"], tflops_burst=p["bf16_tflops"], source="measured")
    return dict(hbm_gbs=6650.0, tflops=1400.0, tflops_burst=1590.0, source="fallback")


def attention_work(w: wl.Workload, depths_sum_plus_rows: int):
    """Algorithmic bytes and flops of one layer of tree attention (all requests)."""
    e = 2 if w.dtype == "bf16" else 4
    byt = 0
    flops = 0
    for P in w.prefix_lens:
        byt += 2 * (P + w.N) * w.Hkv * w.d * e + 2 * w.N * w.Hq * w.d * e + w.N * w.W * 4
        flops += 4 * w.Hq * w.d * (w.N * P)
    flops += 4 * w.Hq * w.d * depths_sum_plus_rows  # visible tree pairs: sum_i (depth_i + 1)
    return byt, flops


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` over all ranks of the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rounds_per_s(requests_per_rank: int, world: int, ms_per_step: float) -> float:
    """Every rank runs an independent replica (no data-path collective): the job's throughput is the
    requests of all ranks over the slowest rank's step time."""
    return requests_per_rank * world / (ms_per_step * 1e-3)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.samples = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            if len(s) < 6:
                continue
            try:
                sm.append(float(s[0]))
                mx = float(s[1])
            except ValueError:
                continue
            for name, v in zip(names, s[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# CPU oracle arm (also the cpu_baseline leg of the GPU arm)
# ------------------------------------------------------------------------------------------------

def oracle_round_seconds(w: wl.Workload, variant: str, attn_pairs: int, seed: int = 0):
    """Time the CPU oracle, as it stands, on one round of `w`: build and accept in full, tree
    attention on `attn_pairs` (row, head) pairs of request 0 / layer 0, scaled to all pairs of all
    requests and layers by pair count.  Returns (seconds per round, description, threads)."""
    from oracle import ddtree_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = 1
    logits = [wl.drafter_logits(w, r, variant, seed) for r in range(w.R)]
    roots = wl.root_tokens(w, seed)
    t0 = time.perf_counter()
    trees = [orc.build(logits[r], w.K, w.B, int(roots[r]), int(w.prefix_lens[r])) for r in range(w.R)]
    t_build = time.perf_counter() - t0

    att = wl.attention_inputs(wl.small_workload(**{**w.__dict__, "R": 1, "prefix_lens": w.prefix_lens[:1]}), 0, seed)
    n = trees[0].n_rows
    rng = np.random.default_rng(seed)
    pairs = [(int(rng.integers(0, n)), int(rng.integers(0, w.Hq))) for _ in range(attn_pairs)]
    q, kc, vc, kt, vt = (att.as_f64(x) for x in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
    t0 = time.perf_counter()
    for (i, h) in pairs:
        orc.tree_attention(q[0], kc, vc, kt[0], vt[0], trees[0].mask, n, rows=[i], heads=[h])
    t_pair = (time.perf_counter() - t0) / max(1, attn_pairs)
    # pairs of the whole round, weighting each request by its key count relative to request 0
    keys0 = w.prefix_lens[0] + n
    total_pairs = sum(trees[r].n_rows * w.Hq * (w.prefix_lens[r] + trees[r].n_rows) / keys0 for r in range(w.R))
    t_attn = t_pair * total_pairs * w.layers

    tl = wl.target_logits(w, trees[0].depth, 0, variant, seed)
    tl64 = wl.bf16_to_f64(tl) if w.dtype == "bf16" else tl.astype(np.float64)
    t0 = time.perf_counter()
    choice = orc.node_argmax(tl64)
    orc.accept_walk(trees[0].token, trees[0].parent, n, choice)
    t_accept = (time.perf_counter() - t0) * w.R
    sample = (f"build and accept in full; tree attention timed on {attn_pairs} random (row, head) pairs of request 0, "
              f"layer 0, scaled by pair count to {w.layers} layers (build {t_build:.3f}s, attention {t_attn:.1f}s "
              f"extrapolated, accept {t_accept:.3f}s)")
    return t_build + t_attn + t_accept, sample, threads


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warmup = args.steps, args.warmup
    # keep the whole run within ~2 minutes: ~25 ms per oracle (row, head) pair at config 1
    budget_s = 100.0 / max(1, steps + warmup)
    pairs = int(min(256, max(8, budget_s / 0.03)))
    times = []
    for i in range(steps + warmup):
        t, sample, threads = oracle_round_seconds(w, args.variant, pairs, seed=0)
        if i >= warmup:
            times.append(t)
    sec = sum(times) / len(times)
    val = w.R / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"config {w.index} ({w.name})", "variant": args.variant, "layers": w.layers,
                   "note": "CPU oracle; every step times a bounded sample and extrapolates attention by pair count"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------

def run_gpu(args, w):
    import torch
    import paper_2604_12989_b200 as dd

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    dd.lib()  # fail loudly if the CUDA library is missing

    bf = w.dtype == "bf16"
    tdt = torch.bfloat16 if bf else torch.float32
    seed = 0
    variant = args.variant

    # ---- inputs: host generators for the logits and layer 0, device RNG for the other layers ----
    logits_h = wl.drafter_logits_batch(w, variant, seed)
    roots_h = wl.root_tokens(w, seed)
    plen_h = np.asarray(w.prefix_lens, np.int32)
    att0 = wl.attention_inputs(w, 0, seed)
    cu_host = att0.cu_prefix.tolist()

    def up(a, bf16=False):
        t = torch.from_numpy(a.view(np.int16) if bf16 else a).to(dev)
        return t.view(torch.bfloat16) if bf16 else t

    logits = up(logits_h)
    roots, plen = up(roots_h), up(plen_h)
    cu = up(att0.cu_prefix)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1234 + rank)
    total_p = int(sum(w.prefix_lens))
    layers = []
    for l in range(w.layers):
        if l == 0:
            layers.append(tuple(up(getattr(att0, n), bf) for n in ("q", "k_cache", "v_cache", "k_tree", "v_tree")))
        else:
            mk = lambda *s: torch.randn(*s, generator=gen, device=dev, dtype=torch.float32).to(tdt)
            layers.append((mk(w.R, w.N, w.Hq, w.d), mk(total_p, w.Hkv, w.d), mk(total_p, w.Hkv, w.d),
                           mk(w.R, w.N, w.Hkv, w.d), mk(w.R, w.N, w.Hkv, w.d)))
    outs = [torch.zeros_like(layers[0][0]) for _ in range(2)]

    # one untimed build gives the tree depths the target-logit generator needs
    tree = dd.ddtree_build(logits, w.K, w.B, roots, plen)
    torch.cuda.synchronize()
    depth_h = tree.node_depth.cpu().numpy()
    target_h = np.stack([wl.target_logits(w, depth_h[r], r, variant, seed) for r in range(w.R)])
    target = up(target_h, bf)

    ws_build = torch.empty(max(256, dd.lib().ddtree_build_workspace_bytes(w.R, w.L, w.V, w.K, w.B)), dtype=torch.uint8, device=dev)
    T = float(args.temperature)
    ws_acc = torch.empty(max(256, (dd.lib().ddtree_accept_sampled_workspace_bytes if T > 0 else
                                   dd.lib().ddtree_accept_workspace_bytes)(w.R, w.B, w.V)), dtype=torch.uint8, device=dev)
    # temperature > 0: one 32-bit random input per row, drawn once with a seeded generator (they are inputs of the
    # call; a serving loop would refresh them on the device every round)
    row_uniform = torch.from_numpy(np.random.default_rng(seed + 17).integers(0, 2 ** 32, (w.R, w.N), dtype=np.uint64)
                                   .astype(np.uint32).view(np.int32)).to(dev)

    def accept_call(tgt, out=None):
        if T > 0:
            return dd.ddtree_accept_sampled(tgt, w.L, tree.node_token, tree.node_parent, tree.n_rows, T, row_uniform,
                                            workspace=ws_acc, out=out)
        return dd.ddtree_accept(tgt, w.L, tree.node_token, tree.node_parent, tree.n_rows, workspace=ws_acc, out=out)

    ws_att = torch.empty(max(256, dd.tree_attention_workspace_bytes(w.R, w.B, w.Hq, w.Hkv, w.d, 1 if bf else 0, cu_host)),
                         dtype=torch.uint8, device=dev)
    acc = accept_call(target)

    def one_round(layer_inputs=layers, tgt=target, lg=logits):
        dd.ddtree_build(lg, w.K, w.B, roots, plen, workspace=ws_build, out=tree)
        for l, (q, kc, vc, kt, vt) in enumerate(layer_inputs):
            dd.ddtree_tree_attention(q, kc, vc, cu_host, cu, kt, vt, tree.anc_mask, tree.n_rows, out=outs[l & 1],
                                     workspace=ws_att)
        accept_call(tgt, acc)

    attn_kernels = 2 if (bf and ws_att.numel() > 256) else 1  # split-KV adds the combine kernel
    launches_per_round = 2 + attn_kernels * w.layers + (4 if T > 0 else 2)

    # ---- capture one round in a CUDA graph (launch-bound otherwise: ~40 host calls per round) ----
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        one_round()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            one_round()
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        graph.replay()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        graph.replay()
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    # keep the GPU busy a little longer so that the clock sampler sees the loaded state
    t_end = time.time() + 0.6
    while time.time() < t_end:
        graph.replay()
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step = max_over_ranks(ms_total / args.steps, dev)
    dd.device_status()

    # ---- per-call duration of the dominant kernel (tree attention), measured live ----------------
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(w.layers)]
    att_ms = []
    for it in range(3 + min(args.steps, 10)):
        dd.ddtree_build(logits, w.K, w.B, roots, plen, workspace=ws_build, out=tree)
        torch.cuda._sleep(6_000_000)  # let the host queue the whole round before the GPU starts on it
        for l, (q, kc, vc, kt, vt) in enumerate(layers):
            evs[l][0].record()
            dd.ddtree_tree_attention(q, kc, vc, cu_host, cu, kt, vt, tree.anc_mask, tree.n_rows, out=outs[l & 1],
                                     workspace=ws_att)
            evs[l][1].record()
        torch.cuda.synchronize()
        if it >= 3:
            att_ms += [a.elapsed_time(b) for a, b in evs]
    att_eager_ms = statistics.mean(att_ms)
    # the same calls in the launch configuration of the timed region: the layers' attention calls alone
    # in a CUDA graph (kernels back to back, each layer with its own L2-cold K/V), replayed between events
    with torch.cuda.stream(stream):
        g_att = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_att, stream=stream):
            for l, (q, kc, vc, kt, vt) in enumerate(layers):
                dd.ddtree_tree_attention(q, kc, vc, cu_host, cu, kt, vt, tree.anc_mask, tree.n_rows, out=outs[l & 1],
                                         workspace=ws_att)
    torch.cuda.synchronize()
    reps = 3 + min(args.steps, 10)
    ga, gb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for it in range(reps):
        if it == 3:
            ga.record()
        g_att.replay()
    gb.record()
    torch.cuda.synchronize()
    att_call_ms = ga.elapsed_time(gb) / ((reps - 3) * w.layers)
    stage_ms = {}
    for name, fn in (("build", lambda: dd.ddtree_build(logits, w.K, w.B, roots, plen, workspace=ws_build, out=tree)),
                     ("accept", lambda: accept_call(target, acc))):
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        ts = []
        for it in range(8):
            flush.fill_(it)  # evict L2 between iterations
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda._sleep(400_000)  # hide the host-side launch latency behind queued work
            a.record(); fn(); b.record()
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(a.elapsed_time(b))
        stage_ms[name] = statistics.mean(ts)
        del flush

    # ---- end to end through the C ABI with host buffers -------------------------------------------
    # Every step's inputs (drafter logits, per-layer Q and tree K/V, target logits) sit in one pinned
    # host arena and cross PCIe in one copy into one of two device arenas; the copy of step i+1 runs on
    # a side stream while step i computes (one captured round per arena); the accept outputs go back to
    # pinned host memory every step.  The KV cache is state and stays in HBM.
    fields = [("logits", logits), ("target", target)]
    for l, (q, kc, vc, kt, vt) in enumerate(layers):
        fields += [(f"q{l}", q), (f"kt{l}", kt), (f"vt{l}", vt)]
    offs, total = {}, 0
    for name, t in fields:
        offs[name] = total
        total += (t.numel() * t.element_size() + 255) // 256 * 256
    h_arena = torch.empty(total, dtype=torch.uint8).pin_memory()
    d_arena = [torch.empty(total, dtype=torch.uint8, device=dev) for _ in range(2)]

    def view(arena, name, like):
        n = like.numel() * like.element_size()
        return arena[offs[name]:offs[name] + n].view(like.dtype).view(like.shape)

    for name, t in fields:
        view(h_arena, name, t).copy_(t.cpu())
    h2d = sum(t.numel() * t.element_size() for _, t in fields)
    h_res = [[torch.empty_like(t, device="cpu").pin_memory() for t in (acc.accept_len, acc.accept_tokens, acc.bonus_token)]
             for _ in range(2)]
    d2h = sum(t.numel() * t.element_size() for t in h_res[0])
    copy_stream = torch.cuda.Stream(device=dev)
    e2e_graphs = []
    with torch.cuda.stream(stream):
        for k in range(2):
            li = [(view(d_arena[k], f"q{l}", q), kc, vc, view(d_arena[k], f"kt{l}", kt), view(d_arena[k], f"vt{l}", vt))
                  for l, (q, kc, vc, kt, vt) in enumerate(layers)]
            args_k = (li, view(d_arena[k], "target", target), view(d_arena[k], "logits", logits))
            d_arena[k].copy_(h_arena, non_blocking=True)
            one_round(*args_k)
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                one_round(*args_k)
                for dst, src in zip(h_res[k], (acc.accept_len, acc.accept_tokens, acc.bonus_token)):
                    dst.copy_(src, non_blocking=True)
            e2e_graphs.append(g)
    torch.cuda.synchronize()
    ready = [torch.cuda.Event() for _ in range(2)]
    done = [torch.cuda.Event() for _ in range(2)]

    def e2e_steps(n):
        for i in range(n):
            k = i & 1
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(done[k])  # arena k is free once the round that used it has finished
                d_arena[k].copy_(h_arena, non_blocking=True)
                ready[k].record(copy_stream)
            with torch.cuda.stream(stream):
                stream.wait_event(ready[k])
                e2e_graphs[k].replay()
                done[k].record(stream)

    with torch.cuda.stream(stream):
        for k in range(2):
            done[k].record(stream)
    e2e_steps(4)
    barrier()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(copy_stream):
        s0.record(copy_stream)
    e2e_steps(args.steps)
    with torch.cuda.stream(stream):
        s1.record(stream)
    barrier()
    assert int(h_res[(args.steps - 1) & 1][0].sum()) == int(acc.accept_len.sum())  # the result was read on the host
    e2e_ms = max_over_ranks(s0.elapsed_time(s1) / args.steps, dev)

    if rank != 0:
        return
    accept_len = acc.accept_len.cpu().numpy()
    n_rows = tree.n_rows.cpu().numpy()
    vis_pairs = int(sum((depth_h[r][:n_rows[r]] + 1).sum() for r in range(w.R)))
    byt, flops = attention_work(w, vis_pairs)
    pk = peaks()
    t_call = att_call_ms * 1e-3
    t_mem, t_mma = byt / (pk["hbm_gbs"] * 1e9), flops / (pk["tflops"] * 1e12)
    if t_mma >= t_mem:
        roof = {"bound": "tensor", "achieved": flops / t_call / 1e12, "peak": pk["tflops"], "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": byt / t_call / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = NCU_TRAFFIC_BYTES.get(w.index)
    roof.update({"kernel": "tree_attention_bf16_kernel (+ split combine), one layer", "peak_source": pk["source"] +
                 " (sustained bf16 GEMM; kernel timed inside a long step)", "algorithmic_bytes": byt,
                 "algorithmic_flops": flops, "us_per_call": att_call_ms * 1e3,
                 "timing": "CUDA events around graph replays that hold only the layers' attention calls (the launch "
                           "configuration of the timed round); issued one by one from the host the same call takes "
                           "%.1f us" % (att_eager_ms * 1e3),
                 "hbm_GBps_at_this_duration": byt / t_call / 1e9, "lower_bound_us": max(t_mem, t_mma) * 1e6})
    e = 4
    logits_gbs = {"build": w.R * w.L * w.V * e / (stage_ms["build"] * 1e-3) / 1e9,
                  "accept": sum(n_rows) * w.V * (2 if bf else 4) / (stage_ms["accept"] * 1e-3) / 1e9}

    probe_s, _, _ = oracle_round_seconds(w, variant, 8)
    per_pair = probe_s / (w.layers * sum(n_rows) * w.Hq) if probe_s > 0 else 1e-3  # rough cost of one pair
    cpu_s, sample, threads = oracle_round_seconds(w, variant, int(min(max(32, 10.0 / max(per_pair, 1e-5)), 2048)))
    line = {
        "metric": METRIC, "value": whole_job_rounds_per_s(w.R, world, ms_per_step), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if bf else "f32", "data": "synthetic",
        "config": {"workload": f"config {w.index} ({w.name})", "variant": variant, "R": w.R, "L": w.L, "V": w.V,
                   "K": w.K, "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "d": w.d, "prefix": list(w.prefix_lens)[:4],
                   "layers": w.layers, "parallelism": f"replicas x{world}",
                   "l2": "inputs larger than L2: every layer has its own K/V cache (%.0f MB per round)" %
                         ((byt * w.layers + w.R * w.L * w.V * 4 + w.R * w.N * w.V * 2) / 1e6),
                   "decoding": "greedy" if T <= 0 else f"temperature {T:g} (ddtree_accept_sampled)",
                   "launch": "one round captured in a CUDA graph and replayed"},
        "tokens_per_s": float((accept_len + 1).sum()) * world / (ms_per_step * 1e-3),
        "accept_len_mean": float(accept_len.mean()),
        "stage_us": {"build": stage_ms["build"] * 1e3, "attention_per_layer": att_call_ms * 1e3,
                     "accept": stage_ms["accept"] * 1e3},
        "logits_pass_GBps": logits_gbs,
        "clocks": clocks,
        "e2e": {"value": whole_job_rounds_per_s(w.R, world, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms, "note": "per round: drafter logits, per-layer Q and tree K/V, target logits "
                "copied from one pinned host arena (copy of step i+1 overlaps the compute of step i); accept outputs "
                "read back every step; the KV cache is state and stays in HBM"},
        "gpu_launches": launches_per_round * args.steps,
        "roofline": roof,
        "cpu_baseline": {"value": w.R / cpu_s, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
    }
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=1, help="workload index (1 = the Qwen3-8B-shaped single request)")
    ap.add_argument("--variant", default="lit", choices=wl.VARIANTS)
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count (profiling small cases only)")
    ap.add_argument("--temperature", type=float, default=0.0,
                    help="0 = the greedy decoding rule (the benchmark's metric); > 0: the verifier walk samples the target's "
                         "choice at that temperature (ddtree_accept_sampled)")
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    args = ap.parse_args()
    w = wl.WORKLOADS[args.config]
    if args.layers > 0:
        import dataclasses
        w = dataclasses.replace(w, layers=args.layers)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_gpu(args, w)


if __name__ == "__main__":
    main()
