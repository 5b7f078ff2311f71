"""GPU parity of ddtree_rope_tree (rotary positional encoding at the tree's position ids, Section 4.4)
against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import ddtree_oracle as orc
from paper_2604_12989_b200 import workloads as wl
from tests import ddtree_cases as cases

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 1e-2}


def build_case(R, B, Hq, Hkv, d, dtype, prefix_lens, seed=0):
    w = wl.small_workload(R=R, L=8, V=600, K=4, B=B, Hq=Hq, Hkv=Hkv, d=d, dtype=dtype, prefix_lens=prefix_lens, index=90)
    logits = cases.drafter_batch(w, "peak")
    trees = cases.oracle_trees(w, logits, wl.root_tokens(w))
    att = wl.attention_inputs(w, 0, seed)
    return w, trees, att


def check(w, trees, att, theta, which=("q", "k")):
    import paper_2604_12989_b200 as dd
    bf = w.dtype == "bf16"
    q = cases.to_torch(att.q, bf) if "q" in which else None
    k = cases.to_torch(att.k_tree, bf) if "k" in which else None
    q0 = None if q is None else q.clone()
    k0 = None if k is None else k.clone()
    pos = torch.from_numpy(np.stack([t.position_ids for t in trees])).cuda()
    n_rows = torch.tensor([t.n_rows for t in trees], dtype=torch.int32).cuda()
    dd.ddtree_rope_tree(q, k, pos, n_rows, theta)
    torch.cuda.synchronize()
    tol = TOL[w.dtype]
    for name, got, before in (("q", q, q0), ("k_tree", k, k0)):
        if got is None:
            continue
        g = got.float().cpu().numpy().astype(np.float64)
        x = att.as_f64(name)
        for r in range(w.R):
            n = trees[r].n_rows
            ref = orc.rope(x[r, :n], trees[r].position_ids[:n], theta)
            err = np.abs(g[r, :n] - ref) / (1 + np.abs(ref))
            assert err.max() <= tol, f"{name} request {r}: {err.max():.3e}"
            assert torch.equal(got[r, n:], before[r, n:])  # padding rows untouched


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d", [64, 128])
def test_rope_small(dtype, d):
    w, trees, att = build_case(3, 40, 8, 2, d, dtype, (0, 77, 5000))
    check(w, trees, att, 1.0e6)


@pytest.mark.parametrize("dtype,d", [("f32", 20), ("bf16", 24), ("f32", 2)])
def test_rope_head_dims_that_do_not_fill_16_byte_vectors(dtype, d):
    w, trees, att = build_case(2, 12, 3, 3, d, dtype, (40, 1000))
    check(w, trees, att, 1.0e4)


def test_rope_long_context_positions_and_small_theta():
    # positions near 10^5 with theta = 10^4: float32 angles would be off by ~10^-2 rad
    w, trees, att = build_case(2, 64, 4, 4, 128, "f32", (99000, 65536))
    check(w, trees, att, 1.0e4)


def test_rope_one_tensor_at_a_time_and_padding_rows():
    w, trees, att = build_case(2, 70, 4, 1, 64, "bf16", (300, 12))
    chain = orc.build(wl.drafter_logits(w, 1, "peak", 0), 1, w.B, 0, 12)  # 9 rows << B + 1
    trees[1] = chain
    check(w, trees, att, 1.0e6, which=("q",))
    check(w, trees, att, 1.0e6, which=("k",))


def test_attention_on_rotated_rows_equals_the_oracle_on_rotated_rows():
    import paper_2604_12989_b200 as dd
    w, trees, att = build_case(1, 64, 8, 2, 128, "bf16", (700,))
    theta = 1.0e6
    q, kc, vc, kt, vt = (cases.to_torch(getattr(att, n), True) for n in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
    pos = torch.from_numpy(trees[0].position_ids[None]).cuda()
    n_rows = torch.tensor([trees[0].n_rows], dtype=torch.int32).cuda()
    mask = torch.from_numpy(trees[0].mask[None].view(np.int32)).cuda()
    dd.ddtree_rope_tree(q, kt, pos, n_rows, theta)
    cu = torch.from_numpy(att.cu_prefix).cuda()
    out = dd.ddtree_tree_attention(q, kc, vc, att.cu_prefix.tolist(), cu, kt, vt, mask, n_rows)
    torch.cuda.synchronize()
    dd.device_status()
    n = trees[0].n_rows
    # the oracle sees what the kernel saw: the rotated rows after rounding to bf16
    qr = q.float().cpu().numpy().astype(np.float64)[0]
    kr = kt.float().cpu().numpy().astype(np.float64)[0]
    ref, _ = orc.tree_attention(qr, att.as_f64("k_cache"), att.as_f64("v_cache"), kr, att.as_f64("v_tree")[0],
                                trees[0].mask, n)
    got = out.float().cpu().numpy().astype(np.float64)[0, :n]
    assert (np.abs(got - ref) / (1 + np.abs(ref))).max() <= 1e-2


def test_rope_argument_errors():
    import paper_2604_12989_b200 as dd
    w, trees, att = build_case(1, 8, 2, 1, 64, "f32", (3,))
    q = cases.to_torch(att.q, False)
    pos = torch.from_numpy(trees[0].position_ids[None]).cuda()
    n_rows = torch.tensor([trees[0].n_rows], dtype=torch.int32).cuda()
    for theta in (0.0, -1.0, float("inf")):
        with pytest.raises(dd.DDTreeError):
            dd.ddtree_rope_tree(q, None, pos, n_rows, theta)
    with pytest.raises(AssertionError):
        dd.ddtree_rope_tree(None, None, pos, n_rows, 1e6)
