"""One whole round (build -> tree attention per layer -> accept -> cache compaction) on the benchmark
workload at full size, captured in a CUDA graph and replayed as bench.py does, against the CPU oracle:
tree arrays, arg-max, acceptance and compacted cache rows bit-exact, attention on sampled (row, head)
pairs within tolerance.  Fewer layers than the benchmark (the layers are independent calls)."""
import numpy as np
import pytest
import torch

from oracle import ddtree_oracle as orc
from paper_2604_12989_b200 import workloads as wl
from tests import ddtree_cases as cases
from tests import test_gpu_attention as ta

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg,layers", [(1, 3), (3, 1)])
def test_round_in_a_cuda_graph_matches_the_oracle(cfg, layers):
    import paper_2604_12989_b200 as dd
    w = wl.WORKLOADS[cfg]
    variant = "peak"
    logits_h = cases.drafter_batch(w, variant)
    roots_h = wl.root_tokens(w)
    trees = cases.oracle_trees(w, logits_h, roots_h)
    tl_h = np.stack([wl.target_logits(w, trees[r].depth, r, variant) for r in range(w.R)])
    atts = [wl.attention_inputs(w, l, 0) for l in range(layers)]

    dev = "cuda"
    logits = torch.from_numpy(logits_h).to(dev)
    roots = torch.from_numpy(roots_h).to(dev)
    plen = torch.tensor(w.prefix_lens, dtype=torch.int32, device=dev)
    target = cases.to_torch(tl_h, True)
    cu_host = atts[0].cu_prefix.tolist()
    cu = torch.from_numpy(atts[0].cu_prefix).to(dev)
    # every request gets a slab with room for the accepted path behind its prefix
    slab = [int(p) + w.L + 1 for p in w.prefix_lens]
    slab_start = np.concatenate([[0], np.cumsum(slab)]).astype(np.int64)
    lay = []
    for att in atts:
        q, kc, vc, kt, vt = (cases.to_torch(getattr(att, n), True) for n in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
        # attention reads the packed cache; compaction writes into slabs that hold the same prefixes
        ks = torch.zeros(int(slab_start[-1]), w.Hkv, w.d, dtype=torch.bfloat16, device=dev)
        vs = torch.zeros_like(ks)
        for r in range(w.R):
            lo, hi = cu_host[r], cu_host[r + 1]
            ks[slab_start[r]:slab_start[r] + hi - lo] = kc[lo:hi]
            vs[slab_start[r]:slab_start[r] + hi - lo] = vc[lo:hi]
        lay.append((q, kc, vc, kt, vt, ks, vs))
    dst = torch.from_numpy(slab_start[:-1] + np.asarray(w.prefix_lens, np.int64)).to(dev)

    ws_b = torch.empty(max(256, dd.lib().ddtree_build_workspace_bytes(w.R, w.L, w.V, w.K, w.B)), dtype=torch.uint8, device=dev)
    ws_a = torch.empty(max(256, dd.lib().ddtree_accept_workspace_bytes(w.R, w.B, w.V)), dtype=torch.uint8, device=dev)
    ws_t = torch.empty(max(256, dd.tree_attention_workspace_bytes(w.R, w.B, w.Hq, w.Hkv, w.d, 1, cu_host)), dtype=torch.uint8, device=dev)
    tree = dd.ddtree_build(logits, w.K, w.B, roots, plen, workspace=ws_b)
    acc = dd.ddtree_accept(target, w.L, tree.node_token, tree.node_parent, tree.n_rows, workspace=ws_a)
    outs = [torch.zeros_like(lay[0][0]) for _ in range(layers)]
    lses = [torch.zeros(w.R, w.N, w.Hq, dtype=torch.float32, device=dev) for _ in range(layers)]

    def one_round():
        dd.ddtree_build(logits, w.K, w.B, roots, plen, workspace=ws_b, out=tree)
        for l, (q, kc, vc, kt, vt, ks, vs) in enumerate(lay):
            dd.ddtree_tree_attention(q, kc, vc, cu_host, cu, kt, vt, tree.anc_mask, tree.n_rows, out=outs[l], lse=lses[l],
                                     workspace=ws_t)
        dd.ddtree_accept(target, w.L, tree.node_token, tree.node_parent, tree.n_rows, workspace=ws_a, out=acc)
        dd.ddtree_kv_compact([x[3] for x in lay], [x[4] for x in lay], [x[5] for x in lay], [x[6] for x in lay], dst,
                             acc.accept_len, acc.accept_nodes)

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        one_round()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            one_round()
    torch.cuda.synchronize()
    # wipe every output, then let only the graph produce them (twice: replays must not depend on leftovers)
    for t in outs + lses + [tree.node_token, tree.anc_mask, acc.accept_len, acc.accept_nodes, acc.node_argmax]:
        t.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    dd.device_status()

    lens = []
    for r in range(w.R):
        cases.tree_arrays_equal(trees[r], tree, r)
        n = trees[r].n_rows
        choice = orc.node_argmax(cases.to_f64(w, tl_h[r]))
        want = orc.accept_walk(trees[r].token, trees[r].parent, n, choice)
        np.testing.assert_array_equal(acc.node_argmax[r].cpu().numpy()[:n], choice[:n])
        assert int(acc.accept_len[r]) == want.accept_len and int(acc.bonus_token[r]) == want.bonus_token
        assert list(acc.accept_nodes[r].cpu().numpy()[:want.accept_len]) == want.nodes
        lens.append(want)
    assert max(x.accept_len for x in lens) >= 1  # the peak variant accepts something
    pairs = ta.sampled_pairs(w, trees, (0,) if cfg == 1 else (), 24, cfg)
    for l, att in enumerate(atts):
        ta.compare(w, att, trees, outs[l].float().cpu().numpy().astype(np.float64), lses[l].cpu().numpy(), pairs)
        for name, slab_t in (("k", lay[l][5]), ("v", lay[l][6])):
            got = slab_t.view(torch.int16).cpu().numpy().view(np.uint16)
            tree_bits = getattr(att, f"{name}_tree")
            cache_bits = getattr(att, f"{name}_cache")
            for r in range(w.R):
                P = w.prefix_lens[r]
                want_slab = np.zeros((slab[r],) + cache_bits.shape[1:], np.uint16)
                want_slab[:P] = cache_bits[cu_host[r]:cu_host[r + 1]]
                want_slab = orc.kv_compact(want_slab, tree_bits[r], P, lens[r].nodes)
                np.testing.assert_array_equal(got[slab_start[r]:slab_start[r + 1]], want_slab)
