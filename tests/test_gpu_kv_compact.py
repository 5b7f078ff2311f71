"""GPU parity of ddtree_kv_compact (end of a round, Section 4.4) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import ddtree_oracle as orc
from paper_2604_12989_b200 import workloads as wl
from tests import ddtree_cases as cases
from tests import test_gpu_attention as ta

pytestmark = pytest.mark.gpu


def walk_with_hits(ct, rng, p_hit=0.85):
    """Target choices that often name a drafted child, and the oracle's walk over them."""
    choice = rng.integers(0, 50, ct.token.shape[0]).astype(np.int32)
    for i in range(ct.n_rows):
        if ct.child_count[i] and rng.random() < p_hit:
            choice[i] = ct.token[ct.first_child[i] + rng.integers(0, ct.child_count[i])]
    return orc.accept_walk(ct.token, ct.parent, ct.n_rows, choice)


def acceptance_tensors(accs, L):
    R = len(accs)
    a_len = torch.tensor([a.accept_len for a in accs], dtype=torch.int32).cuda()
    nodes = np.full((R, L), -1, np.int32)
    for r, a in enumerate(accs):
        nodes[r, :a.accept_len] = a.nodes
    return a_len, torch.from_numpy(nodes).cuda()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_rows_of_the_accepted_path_land_behind_the_prefix(dtype):
    import paper_2604_12989_b200 as dd
    rng = np.random.default_rng(7)
    R, L, B, Hkv, d, layers = 3, 6, 40, 2, 64 if dtype == "f32" else 128, 5
    w = wl.small_workload(R=R, L=L, V=300, K=3, B=B, Hq=4, Hkv=Hkv, d=d, dtype=dtype, prefix_lens=(9, 0, 30), index=41)
    logits = np.stack([wl.drafter_logits(w, r, "peak", 2) for r in range(R)])
    trees = cases.oracle_trees(w, logits, wl.root_tokens(w, 2))
    accs = [walk_with_hits(trees[r], rng, 0.9 if r != 1 else 0.0) for r in range(R)]  # request 1 accepts nothing
    assert accs[1].accept_len == 0 and max(a.accept_len for a in accs) >= 2
    cap = 40  # cache rows per request (slabs of equal size: prefix, then room for L + 1 new rows)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    mk = lambda *s: torch.randn(*s, device="cuda").to(tdt)
    kt, vt = [mk(R, B + 1, Hkv, d) for _ in range(layers)], [mk(R, B + 1, Hkv, d) for _ in range(layers)]
    kc, vc = [mk(R * cap, Hkv, d) for _ in range(layers)], [mk(R * cap, Hkv, d) for _ in range(layers)]
    ref_k, ref_v = [t.float().cpu().numpy() for t in kc], [t.float().cpu().numpy() for t in vc]
    a_len, a_nodes = acceptance_tensors(accs, L)
    dst = torch.tensor([r * cap + w.prefix_lens[r] for r in range(R)], dtype=torch.int64).cuda()
    dd.ddtree_kv_compact(kt, vt, kc, vc, dst, a_len, a_nodes)
    torch.cuda.synchronize()
    for l in range(layers):
        for ref, tree_buf, got in ((ref_k[l], kt[l], kc[l]), (ref_v[l], vt[l], vc[l])):
            want = ref.copy()
            tr = tree_buf.float().cpu().numpy()
            for r in range(R):
                slab = orc.kv_compact(want[r * cap:(r + 1) * cap], tr[r], w.prefix_lens[r], accs[r].nodes)
                want[r * cap:(r + 1) * cap] = slab
            np.testing.assert_array_equal(got.float().cpu().numpy(), want)  # moved rows bit-exact, all others untouched


def test_next_round_attends_to_the_compacted_cache():
    """Two rounds for one request: after accept + compact on the GPU, attention over the extended
    prefix must match the oracle's attention over the oracle's compacted cache."""
    import paper_2604_12989_b200 as dd
    P = 200
    w, att, trees = ta.bf16_case(1, 40, 8, 2, (P,), seed=5)
    acc = next(a for a in (walk_with_hits(trees[0], np.random.default_rng(s), 0.95) for s in range(50)) if a.accept_len >= 3)
    bf = True
    kc, vc, kt, vt = (cases.to_torch(getattr(att, n), bf) for n in ("k_cache", "v_cache", "k_tree", "v_tree"))
    cap = P + w.L + 1
    kc2 = torch.zeros(cap, *kc.shape[1:], dtype=kc.dtype, device="cuda"); kc2[:P] = kc
    vc2 = torch.zeros(cap, *vc.shape[1:], dtype=vc.dtype, device="cuda"); vc2[:P] = vc
    a_len, a_nodes = acceptance_tensors([acc], w.L)
    dd.ddtree_kv_compact([kt], [vt], [kc2], [vc2], torch.tensor([P], dtype=torch.int64).cuda(), a_len, a_nodes)
    P2 = P + acc.accept_len + 1
    # next round: same tree shape and tree K/V stand in for the next block's draft
    w2 = wl.small_workload(**{**w.__dict__, "prefix_lens": (P2,)})
    att2 = wl.attention_inputs(w2, 0, 9)
    att2.k_cache = wl.f32_to_bf16_bits(orc.kv_compact(np.concatenate([wl.bf16_to_f64(att.k_cache), np.zeros((w.L + 1,) + att.k_cache.shape[1:])]),
                                                      wl.bf16_to_f64(att.k_tree)[0], P, acc.nodes)[:P2].astype(np.float32))
    att2.v_cache = wl.f32_to_bf16_bits(orc.kv_compact(np.concatenate([wl.bf16_to_f64(att.v_cache), np.zeros((w.L + 1,) + att.v_cache.shape[1:])]),
                                                      wl.bf16_to_f64(att.v_tree)[0], P, acc.nodes)[:P2].astype(np.float32))
    mask = torch.from_numpy(np.stack([t.mask for t in trees]).view(np.int32)).cuda()
    n_rows = torch.tensor([trees[0].n_rows], dtype=torch.int32).cuda()
    q2, kt2, vt2 = (cases.to_torch(getattr(att2, n), bf) for n in ("q", "k_tree", "v_tree"))
    cu2 = torch.tensor([0, P2], dtype=torch.int32).cuda()
    lse = torch.zeros(1, w.N, w.Hq, dtype=torch.float32, device="cuda")
    out = dd.ddtree_tree_attention(q2, kc2[:P2], vc2[:P2], [0, P2], cu2, kt2, vt2, mask, n_rows, lse=lse)
    torch.cuda.synchronize()
    dd.device_status()
    ta.compare(w2, att2, trees, out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy())
