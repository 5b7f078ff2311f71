#!/usr/bin/env python
"""Benchmark of the DDTree verify round (build + layers x tree attention + accept) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--variant lit|peak] [--configs 0,1,2,3,4]
    python bench.py --impl reference ...      # times the CPU oracle on a bounded sample

One step = one decoding round of the chosen workload: ddtree_build on the drafter logits, one
ddtree_tree_attention call per layer (distinct K/V cache per layer, tree mask taken on the device
from the build of the same step) and ddtree_accept on the target logits.  The headline workload is
config 4 (the largest one that fits a GPU: 70B-shaped, B = 512, prefix 65536, 80 layers); the same JSON
line carries a `per_config` block with every workload of the table timed the same way.  With N > 1
(torchrun) every rank runs an independent replica of the workload (requests are independent; there is no
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
HEADLINE_CONFIG = 4
NOMINAL = {"hbm_gbs": 8000.0, "tflops": 2250.0}  # the figures the benchmark spec names / the dense bf16 data-sheet peak

# dram__bytes_read.sum + dram__bytes_write.sum per launch of tree_attention_bf16_kernel, from the ncu captures
# summarised in profiles/tree_attention_bf16_config{1,2,4}.txt (None: no capture of that workload)
NCU_TRAFFIC_BYTES = {1: 17665024, 2: 73499904, 3: 392809216, 4: 512054272}
MIN_TIMED_SECONDS = 1.0


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


def config_dict(w: wl.Workload, variant: str, world: int, extra=None) -> dict:
    """The workload description both arms print (same keys, so that the two lines can be matched)."""
    d = {"workload": f"config {w.index} ({w.name})", "variant": variant, "R": w.R, "L": w.L, "V": w.V, "K": w.K, "B": w.B,
         "Hq": w.Hq, "Hkv": w.Hkv, "d": w.d, "prefix": list(w.prefix_lens)[:4], "layers": w.layers,
         "parallelism": f"replicas x{world}"}
    d.update(extra or {})
    return d


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,power.draw")

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
            self.samples.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples taken between the two wall-clock times (all of them if not given)."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        return self.summary(t_begin, t_end)

    def summary(self, t_begin=None, t_end=None):
        sm, mx, pw, reasons = [], None, [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, s in list(self.samples):
            if len(s) < 6 or (t_begin is not None and ts < t_begin) or (t_end is not None and ts > t_end):
                continue
            try:
                sm.append(float(s[0]))
                mx = float(s[1])
                if len(s) > 6:
                    pw.append(float(s[6]))
            except ValueError:
                continue
            for name, v in zip(names, s[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm), "power_w": statistics.median(pw) if pw else None,
                "sampled": "inside the timed region"}


# ------------------------------------------------------------------------------------------------
# CPU oracle arm (also the cpu_baseline leg of the GPU arm)
# ------------------------------------------------------------------------------------------------

_POOL_ARGS = None


def _pool_pairs(pairs):
    """Worker: the oracle's tree attention on a list of (row, head) pairs (arguments inherited by fork)."""
    from oracle import ddtree_oracle as orc
    q, kc, vc, kt, vt, mask, n = _POOL_ARGS
    for (i, h) in pairs:
        orc.tree_attention(q, kc, vc, kt, vt, mask, n, rows=[i], heads=[h])
    return len(pairs)


class OracleRound:
    """The CPU oracle, as it stands, on one round of a workload.  Inputs are generated once (not timed); `time`
    runs build and accept in full on one core and tree attention on `attn_pairs` (row, head) pairs of request 0 /
    layer 0, scaled to all pairs of all requests and layers by pair count.  The pairs are spread over forked
    worker processes (one per core this process may run on, at most 32), each with single-threaded BLAS."""

    def __init__(self, w: wl.Workload, variant: str, seed: int = 0, workers: int = 0):
        from oracle import ddtree_oracle as orc
        self.orc, self.w, self.variant, self.seed = orc, w, variant, seed
        self.workers = workers or max(1, min(32, len(os.sched_getaffinity(0))))
        self.logits = [wl.drafter_logits(w, r, variant, seed) for r in range(w.R)]
        self.roots = wl.root_tokens(w, seed)
        self.trees = self.build()
        att = wl.attention_inputs(wl.small_workload(**{**w.__dict__, "R": 1, "prefix_lens": w.prefix_lens[:1]}), 0, seed)
        q, kc, vc, kt, vt = (att.as_f64(x) for x in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
        self.pool_args = (q[0], kc, vc, kt[0], vt[0], self.trees[0].mask, self.trees[0].n_rows)
        tl = wl.target_logits(w, self.trees[0].depth, 0, variant, seed)
        self.tl64 = wl.bf16_to_f64(tl) if w.dtype == "bf16" else tl.astype(np.float64)

    def build(self):
        w = self.w
        return [self.orc.build(self.logits[r], w.K, w.B, int(self.roots[r]), int(w.prefix_lens[r])) for r in range(w.R)]

    def time(self, attn_pairs: int):
        """Returns (seconds per round, description, cores used)."""
        global _POOL_ARGS
        import contextlib
        import multiprocessing as mp
        w, orc, trees = self.w, self.orc, self.trees
        t0 = time.perf_counter()
        self.build()
        t_build = time.perf_counter() - t0
        n = trees[0].n_rows
        rng = np.random.default_rng(self.seed)
        pairs = [(int(rng.integers(0, n)), int(rng.integers(0, w.Hq))) for _ in range(attn_pairs)]
        used = min(self.workers, max(1, attn_pairs))
        chunks = [pairs[k::used] for k in range(used)]
        _POOL_ARGS = self.pool_args
        with contextlib.ExitStack() as stack:
            try:  # one BLAS thread per process: the processes are the parallelism
                from threadpoolctl import threadpool_limits
                stack.enter_context(threadpool_limits(limits=1))
            except Exception:
                pass
            if used > 1:
                with mp.get_context("fork").Pool(used) as pool:
                    pool.map(_pool_pairs, [c[:1] for c in chunks])  # start-up outside the timed region
                    t0 = time.perf_counter()
                    pool.map(_pool_pairs, chunks)
                    t_pairs = time.perf_counter() - t0
            else:
                t0 = time.perf_counter()
                _pool_pairs(pairs)
                t_pairs = time.perf_counter() - t0
        _POOL_ARGS = None
        t_pair = t_pairs / max(1, attn_pairs)  # wall time per pair with `used` cores busy
        # pairs of the whole round, weighting each request by its key count relative to request 0
        keys0 = w.prefix_lens[0] + n
        total_pairs = sum(trees[r].n_rows * w.Hq * (w.prefix_lens[r] + trees[r].n_rows) / keys0 for r in range(w.R))
        t_attn = t_pair * total_pairs * w.layers
        t0 = time.perf_counter()
        choice = orc.node_argmax(self.tl64)
        orc.accept_walk(trees[0].token, trees[0].parent, n, choice)
        t_accept = (time.perf_counter() - t0) * w.R
        sample = (f"build and accept in full on one core; tree attention timed on {attn_pairs} random (row, head) pairs "
                  f"of request 0, layer 0, spread over {used} processes, scaled by pair count to {w.layers} layers "
                  f"(build {t_build:.3f}s, attention {t_attn:.1f}s extrapolated from {t_pairs:.2f}s, accept {t_accept:.3f}s)")
        return t_build + t_attn + t_accept, sample, used

    def pairs_for(self, seconds: float) -> int:
        """How many (row, head) pairs fill about `seconds` of wall time."""
        t, _, used = self.time(2 * self.workers)
        w = self.w
        per_pair = max(1e-6, t / (w.layers * sum(tr.n_rows for tr in self.trees) * w.Hq))  # wall cost of one pair
        return int(min(max(2 * self.workers, seconds / per_pair), 16384))


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    world = int(os.environ.get("WORLD_SIZE", "1"))
    steps, warmup = args.steps, args.warmup
    # keep the whole run within ~2 minutes: every step times a bounded sample of pairs
    oracle = OracleRound(w, args.variant)
    pairs = oracle.pairs_for(75.0 / max(1, steps + warmup))
    times = []
    for i in range(steps + warmup):
        t, sample, cores = oracle.time(pairs)
        if i >= warmup:
            times.append(t)
    sec = sum(times) / len(times)
    val = w.R / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": config_dict(w, args.variant, world, {
            "note": "CPU oracle; every step times a bounded sample and extrapolates attention by pair count"}),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------

def separated_attempts(w, variant, seed):
    """Per request, the first redraw of the drafter logits whose top-B prefix set is separated from the rest by
    1e-3 in log-probability (so that the fp32 build and the fp64 oracle must select the same nodes).  Uses the
    oracle; only the parity leg of the benchmark calls this."""
    from oracle import ddtree_oracle as orc
    out = []
    for r in range(w.R):
        for attempt in range(64):
            x = wl.drafter_logits(w, r, variant, seed, attempt)
            _, lq = orc.top_k(x, w.K)
            if orc.boundary_gap(lq, w.B) >= 1e-3:
                out.append(attempt)
                break
        else:
            out.append(0)
    return out


class RoundBench:
    """Device-resident inputs of one workload and the captured round."""

    def __init__(self, w, dev, variant, temperature, rank, parity):
        import torch
        import paper_2604_12989_b200 as dd
        self.w, self.dev, self.variant, self.T, self.dd, self.torch = w, dev, variant, float(temperature), dd, torch
        bf = self.bf = w.dtype == "bf16"
        tdt = torch.bfloat16 if bf else torch.float32
        seed = self.seed = 0
        # ---- inputs: host generators for the logits and layer 0, device RNG for the other layers ----
        self.attempts = separated_attempts(w, variant, seed) if parity else [0] * w.R
        self.logits_h = wl.drafter_logits_batch(w, variant, seed, self.attempts)
        self.roots_h = wl.root_tokens(w, seed)
        plen_h = np.asarray(w.prefix_lens, np.int32)
        self.att0 = wl.attention_inputs(w, 0, seed)
        self.cu_host = self.att0.cu_prefix.tolist()
        self.logits = self.up(self.logits_h)
        self.roots, self.plen = self.up(self.roots_h), self.up(plen_h)
        self.cu = self.up(self.att0.cu_prefix)
        gen = torch.Generator(device=dev)
        gen.manual_seed(1234 + rank)
        total_p = int(sum(w.prefix_lens))
        self.layers = []
        for l in range(w.layers):
            if l == 0:
                self.layers.append(tuple(self.up(getattr(self.att0, n), bf) for n in ("q", "k_cache", "v_cache", "k_tree", "v_tree")))
            else:
                mk = lambda *s: torch.randn(*s, generator=gen, device=dev, dtype=torch.float32).to(tdt)
                self.layers.append((mk(w.R, w.N, w.Hq, w.d), mk(total_p, w.Hkv, w.d), mk(total_p, w.Hkv, w.d),
                                    mk(w.R, w.N, w.Hkv, w.d), mk(w.R, w.N, w.Hkv, w.d)))
        self.outs = [torch.zeros_like(self.layers[0][0]) for _ in range(2)]
        lib = dd.lib()
        # one untimed build gives the tree depths the target-logit generator needs
        self.tree = dd.ddtree_build(self.logits, w.K, w.B, self.roots, self.plen)
        torch.cuda.synchronize()
        self.depth_h = self.tree.node_depth.cpu().numpy()
        self.target_h = np.stack([wl.target_logits(w, self.depth_h[r], r, variant, seed) for r in range(w.R)])
        self.target = self.up(self.target_h, bf)
        u8 = dict(dtype=torch.uint8, device=dev)
        self.ws_build = torch.empty(max(256, lib.ddtree_build_workspace_bytes(w.R, w.L, w.V, w.K, w.B)), **u8)
        T = self.T
        self.ws_acc = torch.empty(max(256, (lib.ddtree_accept_sampled_workspace_bytes if T > 0 else
                                            lib.ddtree_accept_workspace_bytes)(w.R, w.B, w.V)), **u8)
        # temperature > 0: one 32-bit random input per row, drawn once with a seeded generator (they are inputs of
        # the call; a serving loop would refresh them on the device every round)
        self.row_uniform = torch.from_numpy(np.random.default_rng(seed + 17).integers(0, 2 ** 32, (w.R, w.N), dtype=np.uint64)
                                            .astype(np.uint32).view(np.int32)).to(dev)
        self.ws_att = torch.empty(max(256, dd.tree_attention_workspace_bytes(w.R, w.B, w.Hq, w.Hkv, w.d, 1 if bf else 0,
                                                                             self.cu_host)), **u8)
        self.acc = self.accept_call(self.target)
        # kernels per attention call, as the library plans it for these shapes (a split KV range adds the merge kernel)
        self.attn_kernels = dd.tree_attention_kernel_count(w.R, w.B, w.Hq, w.Hkv, w.d, 1 if bf else 0, self.cu_host)
        self.launches_per_round = 2 + self.attn_kernels * w.layers + (1 if T > 0 else 2)
        self.stream = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(self.stream):
            self.one_round()
            self.stream.synchronize()
            self.graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.graph, stream=self.stream):
                self.one_round()
        torch.cuda.synchronize()

    def up(self, a, bf16=False):
        t = self.torch.from_numpy(a.view(np.int16) if bf16 else a).to(self.dev)
        return t.view(self.torch.bfloat16) if bf16 else t

    def accept_call(self, tgt, out=None):
        w, dd, tree = self.w, self.dd, self.tree
        if self.T > 0:
            # only the walk's outputs are needed: the library draws at the rows the walk stands on
            return dd.ddtree_accept_sampled(tgt, w.L, tree.node_token, tree.node_parent, tree.n_rows, self.T,
                                            self.row_uniform, workspace=self.ws_acc, out=out, all_rows=False)
        return dd.ddtree_accept(tgt, w.L, tree.node_token, tree.node_parent, tree.n_rows, workspace=self.ws_acc, out=out)

    def attention_calls(self, layer_inputs=None):
        dd, tree = self.dd, self.tree
        for l, (q, kc, vc, kt, vt) in enumerate(layer_inputs or self.layers):
            dd.ddtree_tree_attention(q, kc, vc, self.cu_host, self.cu, kt, vt, tree.anc_mask, tree.n_rows,
                                     out=self.outs[l & 1], workspace=self.ws_att)

    def one_round(self, layer_inputs=None, tgt=None, lg=None):
        w = self.w
        self.dd.ddtree_build(self.logits if lg is None else lg, w.K, w.B, self.roots, self.plen,
                             workspace=self.ws_build, out=self.tree)
        self.attention_calls(layer_inputs)
        self.accept_call(self.target if tgt is None else tgt, self.acc)

    # -- measurements ---------------------------------------------------------------------------------
    def time_graph(self, graph, steps, min_seconds, barrier):
        """Replays `graph` in blocks of `steps` (CUDA events around every block) until `min_seconds` of device
        time have passed (at least one block).  Returns (ms per step of the first block, mean over blocks, min
        over blocks, blocks, wall-clock begin and end of the timed region)."""
        torch = self.torch
        blocks = []
        barrier()
        t_begin = time.time()
        while True:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            blocks.append(e0.elapsed_time(e1) / steps)
            if sum(blocks) * steps >= min_seconds * 1e3 or len(blocks) >= 10000:
                break
        t_end = time.time()
        barrier()
        return blocks[0], statistics.mean(blocks), min(blocks), len(blocks), t_begin, t_end

    def attention_only_graph(self):
        torch = self.torch
        with torch.cuda.stream(self.stream):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=self.stream):
                self.attention_calls()
        torch.cuda.synchronize()
        return g

    def stage_times(self):
        """Mean device time of the build and the accept call alone, L2 flushed before every call."""
        torch, w = self.torch, self.w
        out = {}
        for name, fn in (("build", lambda: self.dd.ddtree_build(self.logits, w.K, w.B, self.roots, self.plen,
                                                                 workspace=self.ws_build, out=self.tree)),
                         ("accept", lambda: self.accept_call(self.target, self.acc))):
            flush = torch.empty(256 << 20, dtype=torch.uint8, device=self.dev)
            ts = []
            for it in range(8):
                flush.fill_(it)  # evict L2 between iterations
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda._sleep(400_000)  # hide the host-side launch latency behind queued work
                a.record(); fn(); b.record()
                torch.cuda.synchronize()
                if it >= 3:
                    ts.append(a.elapsed_time(b))
            out[name] = statistics.mean(ts)
            del flush
        return out

    def parity(self, pairs_per_request=4):
        """This run's outputs against the CPU oracle: tree arrays, arg-max / choices, acceptance bit for bit;
        a few (row, head) pairs of layer 0's attention output within the tolerance of the tests."""
        from oracle import ddtree_oracle as orc
        torch, w, dd = self.torch, self.w, self.dd
        tree, acc = self.tree, self.acc
        self.one_round()
        # layer 0's attention output is needed, not the last layer's
        q, kc, vc, kt, vt = self.layers[0]
        out0 = dd.ddtree_tree_attention(q, kc, vc, self.cu_host, self.cu, kt, vt, tree.anc_mask, tree.n_rows, workspace=self.ws_att)
        torch.cuda.synchronize()
        ok_tree = ok_acc = ok_att = True
        worst = 0.0
        rng = np.random.default_rng(5)
        tol = 1e-2 if self.bf else 1e-4
        att = self.att0
        q64, kc64, vc64, kt64, vt64 = (att.as_f64(nm) for nm in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
        for r in range(w.R):
            ct = orc.build(self.logits_h[r], w.K, w.B, int(self.roots_h[r]), int(w.prefix_lens[r]))
            n = ct.n_rows
            ok_tree &= int(tree.n_rows[r]) == n
            for name, want in (("node_token", ct.token), ("node_parent", ct.parent), ("node_depth", ct.depth),
                               ("position_ids", ct.position_ids)):
                ok_tree &= bool(np.array_equal(getattr(tree, name)[r].cpu().numpy(), want))
            ok_tree &= bool(np.array_equal(tree.anc_mask[r].cpu().numpy().view(np.uint32), ct.mask))
            tl = self.target_h[r]
            x = wl.bf16_bits_to_f32(tl) if self.bf else tl  # exact widening: comparisons are the same in fp32 and fp64
            if self.T > 0:
                ks = self.row_uniform[r].cpu().numpy().view(np.uint32).astype(np.uint64)
                choice = orc.node_sampled(x[:n].astype(np.float32), self.T, ks[:n])
            else:
                choice = orc.node_argmax(x)[:n]
            want = orc.accept_walk(ct.token, ct.parent, n, np.concatenate([choice, np.full(w.N - n, -1, np.int32)]))
            if self.T <= 0:  # the sampled walk of the benchmark does not ask for the choice at every row
                ok_acc &= bool(np.array_equal(acc.node_argmax[r].cpu().numpy()[:n], choice))
            ok_acc &= int(acc.accept_len[r]) == want.accept_len and int(acc.bonus_token[r]) == want.bonus_token
            ok_acc &= list(acc.accept_nodes[r].cpu().numpy()[:want.accept_len]) == want.nodes
            lo, hi = att.cu_prefix[r], att.cu_prefix[r + 1]
            oargs = (q64[r], kc64[lo:hi], vc64[lo:hi], kt64[r], vt64[r], ct.mask, n)
            got = out0[r].float().cpu().numpy().astype(np.float64)
            for _ in range(pairs_per_request):
                i, h = int(rng.integers(0, n)), int(rng.integers(0, w.Hq))
                ref, _ = orc.tree_attention(*oargs, rows=[i], heads=[h])
                err = float((np.abs(got[i, h] - ref[0, 0]) / (1 + np.abs(ref[0, 0]))).max())
                worst = max(worst, err)
                ok_att &= err <= tol
        return {"tree_bit_exact": bool(ok_tree), "accept_bit_exact": bool(ok_acc), "attention_within_tol": bool(ok_att),
                "attention_worst_scaled_error": worst, "attention_pairs": pairs_per_request * w.R, "tolerance": tol,
                "ok": bool(ok_tree and ok_acc and ok_att)}


def roofline_of(w, byt, flops, t_call_s, region_s, traffic):
    """Roofline record of one tree-attention call: the bound is the slower of bytes / HBM rate and flops / tensor
    rate at the measured peaks; the tensor peak is the burst figure when the timed region is shorter than a
    second (the chip is not yet at its power cap), else the sustained one."""
    pk = peaks()
    sustained = region_s >= 1.0
    tf = pk["tflops"] if sustained else pk["tflops_burst"]
    t_mem, t_mma = byt / (pk["hbm_gbs"] * 1e9), flops / (tf * 1e12)
    if t_mma >= t_mem:
        roof = {"bound": "tensor", "achieved": flops / t_call_s / 1e12, "peak": tf, "unit": "TFLOP/s",
                "frac_of_nominal": flops / t_call_s / 1e12 / NOMINAL["tflops"], "nominal_peak": NOMINAL["tflops"]}
    else:
        roof = {"bound": "hbm", "achieved": byt / t_call_s / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac_of_nominal": byt / t_call_s / 1e9 / NOMINAL["hbm_gbs"], "nominal_peak": NOMINAL["hbm_gbs"]}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = traffic
    roof.update({"kernel": "bf16 tree attention kernel chosen for the shape (+ split combine), one layer" if w.dtype == "bf16" else
                           "tree_attention_f32_kernel, one layer",
                 "peak_source": "%s (%s; timed region %.2f s)" % (
                     pk["source"], "sustained bf16 GEMM: region of a second or more, the chip sits at its power cap"
                     if sustained else "burst bf16 GEMM: region shorter than a second", region_s),
                 "frac_of_burst_peak": flops / t_call_s / 1e12 / pk["tflops_burst"],
                 "frac_of_sustained_peak": flops / t_call_s / 1e12 / pk["tflops"],
                 "algorithmic_bytes": byt, "algorithmic_flops": flops, "us_per_call": t_call_s * 1e6,
                 "timing": "CUDA events around replays of a graph that holds only the layers' attention calls (the "
                           "launch configuration of the timed round)",
                 "hbm_GBps_at_this_duration": byt / t_call_s / 1e9, "lower_bound_us": max(t_mem, t_mma) * 1e6})
    return roof


def measure_config(w, dev, args, rank, world, barrier, sampler, headline):
    """Everything the JSON line says about one workload.  Returns (record, RoundBench)."""
    import torch
    rb = RoundBench(w, dev, args.variant, args.temperature, rank, parity=not args.no_parity)
    steps = args.steps if headline else max(1, min(args.steps, int(2000 / max(1.0, w.layers))))
    for _ in range(max(3, args.warmup)):
        rb.graph.replay()
    torch.cuda.synchronize()
    first, mean_ms, min_ms, blocks, t0, t1 = rb.time_graph(rb.graph, steps, args.min_seconds, barrier)
    clocks = sampler.summary(t0, t1) if sampler else None
    ms_first = max_over_ranks(first, dev)
    ms_mean = max_over_ranks(mean_ms, dev)
    rb.dd.device_status()
    # the dominant kernel alone, in the launch configuration of the timed round
    g_att = rb.attention_only_graph()
    for _ in range(3):
        g_att.replay()
    a_first, a_mean, a_min, a_blocks, a0, a1 = rb.time_graph(g_att, max(1, steps // 2), args.min_seconds, lambda: torch.cuda.synchronize())
    att_call_ms = a_mean / w.layers
    att_region_s = a_mean * max(1, steps // 2) * a_blocks * 1e-3
    stage_ms = rb.stage_times()
    accept_len = rb.acc.accept_len.cpu().numpy()
    n_rows = rb.tree.n_rows.cpu().numpy()
    vis_pairs = int(sum((rb.depth_h[r][:n_rows[r]] + 1).sum() for r in range(w.R)))
    byt, flops = attention_work(w, vis_pairs)
    roof = roofline_of(w, byt, flops, att_call_ms * 1e-3, att_region_s, NCU_TRAFFIC_BYTES.get(w.index))
    pk = peaks()
    e_t = 2 if rb.bf else 4
    gbs_build = w.R * w.L * w.V * 4 / (stage_ms["build"] * 1e-3) / 1e9
    gbs_accept = float(sum(n_rows)) * w.V * e_t / (stage_ms["accept"] * 1e-3) / 1e9
    rec = {
        "workload": f"config {w.index} ({w.name})",
        "ms_per_step": ms_mean, "ms_per_step_min_block": min_ms, "ms_per_step_first_block": ms_first,
        "timed": {"steps_per_block": steps, "blocks": blocks, "seconds": mean_ms * steps * blocks * 1e-3},
        "rounds_per_s": whole_job_rounds_per_s(w.R, world, ms_mean),
        "tokens_per_s": float((accept_len + 1).sum()) * world / (ms_mean * 1e-3),
        "tokens_per_round": float((accept_len + 1).sum()),
        "accept_len_mean": float(accept_len.mean()),
        "stage_us": {"build": stage_ms["build"] * 1e3, "attention_per_layer": att_call_ms * 1e3,
                     "attention_per_layer_min_block": a_min / w.layers * 1e3, "accept": stage_ms["accept"] * 1e3},
        "logits_pass_GBps": {"build_stage": gbs_build, "accept_stage": gbs_accept,
                             "build_frac_of_measured_hbm": gbs_build / pk["hbm_gbs"], "build_frac_of_8TBps": gbs_build / NOMINAL["hbm_gbs"],
                             "accept_frac_of_measured_hbm": gbs_accept / pk["hbm_gbs"], "accept_frac_of_8TBps": gbs_accept / NOMINAL["hbm_gbs"],
                             "note": "whole stage (logits pass + tree kernel / walk kernel) over the logits bytes; the passes "
                                     "alone are in profiles/"},
        "roofline": roof, "clocks": clocks,
        "gpu_launches_per_round": rb.launches_per_round,
    }
    if not args.no_parity and rank == 0:
        rec["parity"] = rb.parity()
    return rec, rb, steps


def e2e_measure(rb, args, barrier):
    """End to end through the C ABI with host buffers.  Every step's inputs (drafter logits, per-layer Q and tree
    K/V, target logits) sit in one pinned host arena and cross PCIe in one copy into one of two device arenas;
    the copy of step i+1 runs on a side stream while step i computes (one captured round per arena); the accept
    outputs go back to pinned host memory every step.  The KV cache is state and stays in HBM."""
    import torch
    w, dev, stream, acc = rb.w, rb.dev, rb.stream, rb.acc
    fields = [("logits", rb.logits), ("target", rb.target)]
    for l, (q, kc, vc, kt, vt) in enumerate(rb.layers):
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
                  for l, (q, kc, vc, kt, vt) in enumerate(rb.layers)]
            args_k = (li, view(d_arena[k], "target", rb.target), view(d_arena[k], "logits", rb.logits))
            d_arena[k].copy_(h_arena, non_blocking=True)
            rb.one_round(*args_k)
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                rb.one_round(*args_k)
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
    return max_over_ranks(s0.elapsed_time(s1) / args.steps, dev), h2d, d2h


def run_gpu(args):
    import torch
    import paper_2604_12989_b200 as dd

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    # The timed CPU oracle runs first, before this process touches CUDA: its (row, head) pairs are spread over
    # forked worker processes, and a process should fork before it holds a CUDA context.
    cpu_line = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        w0 = wl.WORKLOADS[args.config]
        if args.layers > 0:
            import dataclasses
            w0 = dataclasses.replace(w0, layers=args.layers)
        oracle = OracleRound(w0, args.variant)
        cpu_s, sample, cores = oracle.time(oracle.pairs_for(12.0))
        del oracle
        cpu_line = {"value": w0.R / cpu_s, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    dd.lib()  # fail loudly if the CUDA library is missing

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.25)

    head_index = args.config
    per_config = {}
    others = [c for c in args.configs if c != head_index]
    # the other workloads first (each frees its tensors before the next one starts), the headline last
    for c in others:
        w = wl.WORKLOADS[c]
        rec, rb, _ = measure_config(w, dev, args, rank, world, barrier, sampler, headline=False)
        per_config[str(c)] = rec
        del rb
        torch.cuda.empty_cache()
    w = wl.WORKLOADS[head_index]
    if args.layers > 0:
        import dataclasses
        w = dataclasses.replace(w, layers=args.layers)
    head, rb, steps = measure_config(w, dev, args, rank, world, barrier, sampler, headline=True)
    per_config[str(head_index)] = head
    e2e_ms, h2d, d2h = e2e_measure(rb, args, barrier)
    if sampler:
        sampler.stop()

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return
    T = float(args.temperature)
    byt = head["roofline"]["algorithmic_bytes"]
    ms_per_step = head["ms_per_step_first_block"]  # exactly `steps` steps after the warm-up, as the contract asks
    line = {
        "metric": METRIC, "value": whole_job_rounds_per_s(w.R, world, ms_per_step), "unit": UNIT, "n_gpus": world,
        "steps": steps, "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
        "config": config_dict(w, args.variant, world, {
            "l2": "inputs larger than L2: every layer has its own K/V cache (%.0f MB per round)" %
                  ((byt * w.layers + w.R * w.L * w.V * 4 + w.R * w.N * w.V * 2) / 1e6),
            "decoding": "greedy" if T <= 0 else f"temperature {T:g} (ddtree_accept_sampled)",
            "launch": "one round captured in a CUDA graph and replayed",
            "why_this_workload": "the largest workload of the table that fits one GPU; the others are in per_config"}),
        "ms_per_step_mean_over_%.1fs" % head["timed"]["seconds"]: head["ms_per_step"],
        "tokens_per_s": head["tokens_per_round"] * world / (ms_per_step * 1e-3),
        "accept_len_mean": head["accept_len_mean"],
        "stage_us": head["stage_us"],
        "logits_pass_GBps": head["logits_pass_GBps"],
        "clocks": head["clocks"],
        "e2e": {"value": whole_job_rounds_per_s(w.R, world, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
                "note": "per round: drafter logits, per-layer Q and tree K/V, target logits copied from one pinned host "
                        "arena (copy of step i+1 overlaps the compute of step i); accept outputs read back every step; "
                        "the KV cache is state and stays in HBM"},
        "gpu_launches": head["gpu_launches_per_round"] * steps,
        "roofline": head["roofline"],
        "parity": head.get("parity"),
        "per_config": per_config,
        "targets": {
            "tree_attention_frac_of_binding_roofline_ge_0.60": {k: v["roofline"]["frac"] >= 0.60 for k, v in per_config.items()},
            "note": "north_star asks 0.60 of the binding roofline for tree attention and 0.70 of HBM peak for the logits "
                    "passes; fractions of the measured and of the nominal peaks are both in `roofline` / `logits_pass_GBps`"},
        "cpu_baseline": cpu_line,
    }
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=12)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=HEADLINE_CONFIG,
                    help="headline workload (4 = the 70B-shaped long-context request, the largest that fits one GPU)")
    ap.add_argument("--configs", default="0,1,2,3,4", help="workloads of the per_config block (comma separated)")
    ap.add_argument("--variant", default="peak", choices=wl.VARIANTS,
                    help="input recipe: `peak` gives accepted paths of several tokens, `lit` (the boost as written) accepts nothing")
    ap.add_argument("--layers", type=int, default=0, help="override the headline workload's layer count (profiling small cases only)")
    ap.add_argument("--temperature", type=float, default=0.0,
                    help="0 = the greedy decoding rule (the benchmark's metric); > 0: the verifier walk samples the target's "
                         "choice at that temperature (ddtree_accept_sampled)")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS,
                    help="every workload's timed regions repeat their block of steps until this much device time has passed "
                         "(0: one block; profiling runs)")
    ap.add_argument("--no-parity", action="store_true", help="skip the oracle comparison of every workload's outputs")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the timed CPU oracle (profiling runs)")
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    args = ap.parse_args()
    args.configs = sorted({int(c) for c in str(args.configs).split(",") if c != ""} | {args.config})
    if args.impl == "reference":
        w = wl.WORKLOADS[args.config]
        if args.layers > 0:
            import dataclasses
            w = dataclasses.replace(w, layers=args.layers)
        run_reference(args, w)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
