"""Context measurement, not part of the library's path: the attention of a verification pass the way the paper
runs it (Appendix B: PyTorch scaled-dot-product attention with an explicit tree mask) beside ddtree_tree_attention,
on the same synthetic layers of the benchmark workloads and the same GPU.

    python -m paper_2604_12989_b200.sdpa_context [--configs 1,2,3,4]

Per layer and request the library call gets q [1, Hq, N, d], k / v [1, Hkv, P + N, d] (the tree's keys appended to
the request's cached prefix, as a Hugging Face decoder does) and a boolean mask [N, P + N] (prefix columns all true,
tree columns from the ancestor bitmask); grouped-query attention through `enable_gqa`.  Building k / v / mask is not
timed.  Both sides: a CUDA graph over `layers` layers with distinct K/V (inputs larger than L2), CUDA events."""
from __future__ import annotations

import argparse

import numpy as np


def measure(ci: int, layers: int, reps: int = 5):
    import torch
    import torch.nn.functional as F
    import paper_2604_12989_b200 as dd
    from paper_2604_12989_b200 import workloads as wl

    dev = torch.device("cuda")
    w = wl.WORKLOADS[ci]
    mk = lambda *s: torch.randn(*s, device=dev).to(torch.bfloat16)
    P = sum(w.prefix_lens)
    L = [(mk(w.R, w.N, w.Hq, w.d), mk(P, w.Hkv, w.d), mk(P, w.Hkv, w.d), mk(w.R, w.N, w.Hkv, w.d), mk(w.R, w.N, w.Hkv, w.d))
         for _ in range(layers)]
    logits = torch.from_numpy(wl.drafter_logits_batch(w, "peak")).to(dev)
    tree = dd.ddtree_build(logits, w.K, w.B, torch.zeros(w.R, dtype=torch.int32, device=dev),
                           torch.tensor(w.prefix_lens, dtype=torch.int32, device=dev))
    cu_np = np.asarray(w.cu_prefix)
    cu, cuh = torch.from_numpy(cu_np).to(dev), cu_np.tolist()
    out = torch.zeros_like(L[0][0])
    ws = torch.empty(max(256, dd.tree_attention_workspace_bytes(w.R, w.B, w.Hq, w.Hkv, w.d, 1, cuh)), dtype=torch.uint8, device=dev)

    # the library call's inputs: per layer and request, K/V = prefix + tree, and the dense boolean mask
    bits = tree.anc_mask.cpu().numpy().view(np.uint32)                     # [R, N, W]
    tree_vis = ((bits[:, :, :, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(w.R, w.N, -1)[:, :, :w.N].astype(bool)
    masks, sd = [], []
    for r in range(w.R):
        Pr = w.prefix_lens[r]
        m = np.concatenate([np.ones((w.N, Pr), bool), tree_vis[r]], axis=1)
        masks.append(torch.from_numpy(m).to(dev))
    for l in L:
        per_req = []
        for r in range(w.R):
            lo, hi = cuh[r], cuh[r + 1]
            k = torch.cat([l[1][lo:hi], l[3][r]]).transpose(0, 1)[None].contiguous()   # [1, Hkv, P + N, d]
            v = torch.cat([l[2][lo:hi], l[4][r]]).transpose(0, 1)[None].contiguous()
            q = l[0][r].transpose(0, 1)[None].contiguous()                             # [1, Hq, N, d]
            per_req.append((q, k, v))
        sd.append(per_req)

    def ours():
        for l in L:
            dd.ddtree_tree_attention(l[0], l[1], l[2], cuh, cu, l[3], l[4], tree.anc_mask, tree.n_rows, out=out, workspace=ws)

    def library():
        for per_req in sd:
            for r, (q, k, v) in enumerate(per_req):
                F.scaled_dot_product_attention(q, k, v, attn_mask=masks[r], enable_gqa=True)

    def timed(fn):
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            fn()
            st.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=st):
                fn()
        torch.cuda.synchronize()
        for _ in range(3):
            g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (reps * layers)

    # same answer first (request 0, all rows of the tree)
    ours()
    q, k, v = sd[-1][0]
    ref = F.scaled_dot_product_attention(q, k, v, attn_mask=masks[0], enable_gqa=True)[0].transpose(0, 1).float()
    n0 = int(tree.n_rows[0])
    err = ((out[0, :n0].float() - ref[:n0]).abs() / (1 + ref[:n0].abs())).max().item()
    t_ours, t_lib = timed(ours), timed(library)
    dd.device_status()
    return {"config": ci, "layers": layers, "us_per_layer_ddtree": t_ours, "us_per_layer_sdpa_masked": t_lib,
            "ratio": t_lib / t_ours, "max_scaled_difference": err}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="1,2,3,4")
    a = ap.parse_args()
    for ci in (int(x) for x in a.configs.split(",")):
        r = measure(ci, layers=12 if ci != 4 else 4)
        print("config %d: ddtree_tree_attention %8.1f us/layer   torch SDPA with explicit tree mask %9.1f us/layer   x%.1f   "
              "(largest scaled difference between the two outputs %.1e)" % (ci, r["us_per_layer_ddtree"], r["us_per_layer_sdpa_masked"],
                                                                          r["ratio"], r["max_scaled_difference"]), flush=True)


if __name__ == "__main__":
    main()
