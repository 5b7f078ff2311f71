"""Synthetic closed loop over several decoding rounds for a range of node budgets (the trade-off the
paper studies in Section 5.3 and Figure 3: a larger tree raises the acceptance length but also the
cost of the verifier pass).

    python -m paper_2604_12989_b200.budget_sweep [--budgets 16,32,...] [--rounds 24] [--layers 36]

One request (the paper runs batch size 1).  Every round: drafter logits for the next block and, once
the tree is built, target logits for its nodes are drawn on the device (noise plus a boost on a hidden
true token per depth; the drafter's boost is drawn per position around the largest of the V noise draws
(mean --draft-boost0 sigmas, falling by --draft-slope per depth, spread --draft-jitter), so at most
positions the true token is the drafter's first choice, and where it is not it usually sits among the
next few ranks: a larger tree catches more of those; the target always prefers the true token); then,
timed with CUDA events,
ddtree_build -> one ddtree_tree_attention per layer (after ddtree_rope_tree with --rope-theta) -> ddtree_accept
(ddtree_accept_sampled with --temperature) -> ddtree_kv_compact, after which
the accepted path is part of the KV cache and the prefix has grown by accept_len + 1.  There is no
model behind the logits, so the acceptance lengths are those of the recipe, not of Qwen3; what the
sweep shows on this GPU is how the cost of a round grows with the budget and where tokens/s peaks
for a given acceptance curve.  The rest of a verifier pass (the target's weight-bound layers) is not
run; `--model-params` adds it as a model, max(weight bytes / HBM rate, 2 x params x rows / tensor rate)
per round, so that the budget at which tokens/s peaks can be read off for a target of that size
(clearly a model, printed in a column of its own).  Prints one line per budget and a JSON summary."""
from __future__ import annotations

import argparse
import json
import statistics

import numpy as np


def run(budgets, rounds, layers, prefix, seed=0, draft_boost0=5.0, draft_slope=0.05, temperature=0.0, rope_theta=0.0,
        draft_jitter=0.6, model_params=0.0, hbm_gbs=6521.0, tflops=1381.0):
    import torch
    import paper_2604_12989_b200 as dd
    from paper_2604_12989_b200 import workloads as wl

    dev = torch.device("cuda")
    dd.lib()
    out = []
    for B in budgets:
        K = 8 if B <= 64 else 16
        w = wl.small_workload(R=1, L=16, V=151936, K=K, B=B, Hq=32, Hkv=8, d=128, dtype="bf16",
                              prefix_lens=(prefix,), layers=layers, noise=3.0, boost0=8.0, boost_slope=0.25, index=60)
        gen = torch.Generator(device=dev)
        gen.manual_seed(seed * 1000 + B)
        cap = prefix + rounds * (w.L + 1)
        mk = lambda *s: torch.randn(*s, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        kc = [mk(cap, w.Hkv, w.d) for _ in range(layers)]
        vc = [mk(cap, w.Hkv, w.d) for _ in range(layers)]
        qs = [mk(1, w.N, w.Hq, w.d) for _ in range(layers)]
        kt = [mk(1, w.N, w.Hkv, w.d) for _ in range(layers)]
        vt = [mk(1, w.N, w.Hkv, w.d) for _ in range(layers)]
        outs = [torch.empty_like(qs[0]) for _ in range(2)]
        depth_tab = np.arange(1, w.L + 2)
        boost = torch.from_numpy(wl._boost(w, 0, depth_tab, "peak", seed)).to(dev)           # target: boost of depth 1..L+1
        draft_mean = torch.from_numpy(((draft_boost0 - draft_slope * depth_tab) * w.noise).astype(np.float32)).to(dev)
        ws_b = torch.empty(max(256, dd.lib().ddtree_build_workspace_bytes(1, w.L, w.V, K, B)), dtype=torch.uint8, device=dev)
        ws_a = torch.empty(max(256, dd.lib().ddtree_accept_sampled_workspace_bytes(1, B, w.V)), dtype=torch.uint8, device=dev)
        roots = torch.zeros(1, dtype=torch.int32, device=dev)
        P = prefix
        times, lens, rows = [], [], []
        tree = acc = None
        for rnd in range(rounds + 2):                                                        # two warm-up rounds
            y = torch.randint(0, w.V, (w.L + 1,), generator=gen, device=dev)                # hidden true tokens of this block
            logits = torch.randn(1, w.L, w.V, generator=gen, device=dev) * w.noise
            draft_boost = draft_mean[:w.L] + draft_jitter * w.noise * torch.randn(w.L, generator=gen, device=dev)
            logits[0, torch.arange(w.L, device=dev), y[:w.L]] = draft_boost  # the true token's logit itself, not an offset
            plen = torch.tensor([P], dtype=torch.int32, device=dev)
            cu_host = [0, P]
            cu = torch.tensor(cu_host, dtype=torch.int32, device=dev)
            ws_t = torch.empty(max(256, dd.tree_attention_workspace_bytes(1, B, w.Hq, w.Hkv, w.d, 1, cu_host)),
                               dtype=torch.uint8, device=dev)
            # target logits need the depths of the tree: build once untimed, as the target model would sit in between
            tree = dd.ddtree_build(logits, K, B, roots, plen, workspace=ws_b, out=tree)
            depth = tree.node_depth[0].long().clamp(min=0)
            target = (torch.randn(w.N, w.V, generator=gen, device=dev) * w.noise)
            target[torch.arange(w.N, device=dev), y[depth]] += boost[depth]
            target = target.to(torch.bfloat16)[None]
            dst = torch.tensor([P], dtype=torch.int64, device=dev)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda._sleep(8_000_000)                                                     # let the host queue the round
            e0.record()
            dd.ddtree_build(logits, K, B, roots, plen, workspace=ws_b, out=tree)
            for l in range(layers):
                if rope_theta > 0:  # the tree's Q / K rows of this layer at their position ids (in place: the synthetic
                    dd.ddtree_rope_tree(qs[l], kt[l], tree.position_ids, tree.n_rows, rope_theta)  # rows are reused as they are)
                dd.ddtree_tree_attention(qs[l], kc[l][:P], vc[l][:P], cu_host, cu, kt[l], vt[l], tree.anc_mask, tree.n_rows,
                                         out=outs[l & 1], workspace=ws_t)
            if temperature > 0:
                uni = torch.randint(-2 ** 31, 2 ** 31 - 1, (1, w.N), generator=gen, device=dev, dtype=torch.int32)
                acc = dd.ddtree_accept_sampled(target, w.L, tree.node_token, tree.node_parent, tree.n_rows, temperature, uni,
                                               workspace=ws_a, out=acc, all_rows=False)
            else:
                acc = dd.ddtree_accept(target, w.L, tree.node_token, tree.node_parent, tree.n_rows, workspace=ws_a, out=acc)
            dd.ddtree_kv_compact(kt, vt, kc, vc, dst, acc.accept_len, acc.accept_nodes)
            e1.record()
            torch.cuda.synchronize()
            a = int(acc.accept_len[0])
            roots = acc.bonus_token.clone()
            if rnd >= 2:
                times.append(e0.elapsed_time(e1))
                lens.append(a)
                rows.append(int(tree.n_rows[0]))
            P += a + 1
        dd.device_status()
        ms = statistics.mean(times)
        tau = statistics.mean(lens) + 1
        rec = {"B": B, "K": K, "rows": statistics.mean(rows), "ms_per_round": ms, "tau": tau, "tokens_per_s": tau / (ms * 1e-3)}
        if model_params > 0:  # the target's dense layers, modelled: bf16 weights read once, or the GEMM flops of all rows
            model_ms = max(2.0 * model_params / (hbm_gbs * 1e9), 2.0 * model_params * (B + 1) / (tflops * 1e12)) * 1e3
            rec["modelled_verifier_ms"] = model_ms
            rec["tokens_per_s_with_modelled_verifier"] = tau / ((ms + model_ms) * 1e-3)
        out.append(rec)
        extra = (f"  | + modelled verifier {rec['modelled_verifier_ms']:6.2f} ms: {rec['tokens_per_s_with_modelled_verifier']:7.0f} tokens/s"
                 if model_params > 0 else "")
        print(f"B={B:5d} K={K:2d} rows={rec['rows']:7.1f}  round {ms:7.3f} ms  tau {tau:5.2f}  {rec['tokens_per_s']:9.0f} tokens/s{extra}", flush=True)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--budgets", default="16,32,64,128,256,512,1024")
    ap.add_argument("--rounds", type=int, default=24)
    ap.add_argument("--layers", type=int, default=36)
    ap.add_argument("--prefix", type=int, default=4096)
    ap.add_argument("--draft-boost0", type=float, default=5.0, help="mean drafter logit of the true token at depth 0, in noise sigmas")
    ap.add_argument("--draft-slope", type=float, default=0.05, help="decrease of that mean per depth, in noise sigmas")
    ap.add_argument("--draft-jitter", type=float, default=0.6, help="spread of the true token's drafter logit, in noise sigmas")
    ap.add_argument("--model-params", type=float, default=0.0,
                    help="> 0: add a modelled verifier pass of a dense bf16 target with this many parameters to every round")
    ap.add_argument("--temperature", type=float, default=0.0, help="> 0: the walk samples the target's choice (ddtree_accept_sampled)")
    ap.add_argument("--rope-theta", type=float, default=0.0, help="> 0: rotate every layer's tree Q / K rows first (ddtree_rope_tree)")
    a = ap.parse_args()
    res = run([int(x) for x in a.budgets.split(",")], a.rounds, a.layers, a.prefix, 0, a.draft_boost0, a.draft_slope,
              a.temperature, a.rope_theta, a.draft_jitter, a.model_params)
    print(json.dumps({"sweep": res, "layers": a.layers, "prefix": a.prefix, "rounds": a.rounds, "temperature": a.temperature,
                      "rope_theta": a.rope_theta, "draft": [a.draft_boost0, a.draft_slope, a.draft_jitter], "model_params": a.model_params,
                      "launch": "eager (host-issued calls)"}))


if __name__ == "__main__":
    main()
