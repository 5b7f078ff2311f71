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


# ---------------------------------------------------------------------------------------------
# ddtree_tree_attention_rope: the same encoding applied inside the attention kernel's load path
# ---------------------------------------------------------------------------------------------

def fused_vs_oracle(w, trees, att, theta, softmax_scale=0.0):
    """The fused call on unrotated rows against the oracle's attention over the oracle's rotated rows (rounded to
    bf16 as the kernel rounds them before its products)."""
    import paper_2604_12989_b200 as dd
    q, kc, vc, kt, vt = (cases.to_torch(getattr(att, n), True) for n in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
    q0, kt0 = q.clone(), kt.clone()
    pos = torch.from_numpy(np.stack([t.position_ids for t in trees])).cuda()
    n_rows = torch.tensor([t.n_rows for t in trees], dtype=torch.int32).cuda()
    mask = torch.from_numpy(np.stack([t.mask for t in trees]).view(np.int32)).cuda()
    cu = torch.from_numpy(att.cu_prefix).cuda()
    lse = torch.zeros(w.R, w.N, w.Hq, dtype=torch.float32, device="cuda")
    out = dd.ddtree_tree_attention_rope(q, kc, vc, att.cu_prefix.tolist(), cu, kt, vt, mask, n_rows, pos, theta, lse=lse,
                                        softmax_scale=softmax_scale)
    torch.cuda.synchronize()
    dd.device_status()
    assert torch.equal(q, q0) and torch.equal(kt, kt0)  # inputs are not modified
    got = out.float().cpu().numpy().astype(np.float64)
    worst = 0.0
    for r in range(w.R):
        n = trees[r].n_rows
        lo, hi = att.cu_prefix[r], att.cu_prefix[r + 1]
        qr = np.zeros_like(att.as_f64("q")[r])
        kr = np.zeros_like(att.as_f64("k_tree")[r])
        qr[:n] = wl.bf16_to_f64(wl.f32_to_bf16_bits(orc.rope(att.as_f64("q")[r, :n], trees[r].position_ids[:n], theta).astype(np.float32)))
        kr[:n] = wl.bf16_to_f64(wl.f32_to_bf16_bits(orc.rope(att.as_f64("k_tree")[r, :n], trees[r].position_ids[:n], theta).astype(np.float32)))
        kw = {} if softmax_scale == 0.0 else {"scale": softmax_scale}
        ref, ref_lse = orc.tree_attention(qr, att.as_f64("k_cache")[lo:hi], att.as_f64("v_cache")[lo:hi], kr,
                                          att.as_f64("v_tree")[r], trees[r].mask, n, **kw)
        err = np.abs(got[r, :n] - ref) / (1 + np.abs(ref))
        worst = max(worst, err.max())
        assert err.max() <= 1e-2, f"request {r}: {err.max():.3e}"
        np.testing.assert_allclose(lse[r, :n].cpu().numpy(), ref_lse, atol=2e-2, rtol=1e-2)
        assert (got[r, n:] == 0).all()
    return worst


@pytest.mark.parametrize("R,B,Hq,Hkv,prefix", [
    (1, 64, 8, 2, (700,)),            # split KV range, one tree tile, 4 rows left over (no short-tile path in this variant)
    (2, 200, 4, 1, (260, 100000)),     # two tree tiles, a long-context position (angles need the double-precision reduction)
    (3, 40, 16, 4, (0, 129, 5)),       # no cached context: every key tile is a rotated tree tile
    (40, 31, 16, 4, None),             # a batch that fills the GPU: unsplit
    (1, 1024, 16, 1, (300,)),          # the largest tree: nine tree tiles
])
def test_fused_rope_attention_equals_the_oracle_on_rotated_rows(R, B, Hq, Hkv, prefix):
    if prefix is None:
        prefix = tuple(int(x) for x in np.random.default_rng(3).integers(1, 400, R))
    w, trees, att = build_case(R, B, Hq, Hkv, 128, "bf16", prefix)
    fused_vs_oracle(w, trees, att, 1.0e6)


def test_fused_rope_equals_the_separate_pass():
    """ddtree_rope_tree on copies followed by ddtree_tree_attention, against the fused call: the same rotated
    bf16 rows enter the same products, so the outputs agree to within the rounding of the rotation itself."""
    import paper_2604_12989_b200 as dd
    w, trees, att = build_case(2, 100, 8, 2, 128, "bf16", (900, 77))
    theta = 1.0e4
    q, kc, vc, kt, vt = (cases.to_torch(getattr(att, n), True) for n in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
    pos = torch.from_numpy(np.stack([t.position_ids for t in trees])).cuda()
    n_rows = torch.tensor([t.n_rows for t in trees], dtype=torch.int32).cuda()
    mask = torch.from_numpy(np.stack([t.mask for t in trees]).view(np.int32)).cuda()
    cu = torch.from_numpy(att.cu_prefix).cuda()
    fused = dd.ddtree_tree_attention_rope(q, kc, vc, att.cu_prefix.tolist(), cu, kt, vt, mask, n_rows, pos, theta)
    q2, kt2 = q.clone(), kt.clone()
    dd.ddtree_rope_tree(q2, kt2, pos, n_rows, theta)
    sep = dd.ddtree_tree_attention(q2, kc, vc, att.cu_prefix.tolist(), cu, kt2, vt, mask, n_rows)
    torch.cuda.synchronize()
    dd.device_status()
    a, b = fused.float(), sep.float()
    assert float(((a - b).abs() / (1 + b.abs())).max()) <= 4e-3


def test_fused_rope_argument_errors():
    import paper_2604_12989_b200 as dd
    w, trees, att = build_case(1, 8, 2, 1, 128, "bf16", (3,))
    q, kc, vc, kt, vt = (cases.to_torch(getattr(att, n), True) for n in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
    pos = torch.from_numpy(trees[0].position_ids[None]).cuda()
    n_rows = torch.tensor([trees[0].n_rows], dtype=torch.int32).cuda()
    mask = torch.from_numpy(trees[0].mask[None].view(np.int32)).cuda()
    cu = torch.from_numpy(att.cu_prefix).cuda()
    for theta in (0.0, -1.0, float("inf")):
        with pytest.raises(dd.DDTreeError):
            dd.ddtree_tree_attention_rope(q, kc, vc, att.cu_prefix.tolist(), cu, kt, vt, mask, n_rows, pos, theta)
    with pytest.raises(dd.DDTreeError) as e:  # fp32 has no fused variant
        dd.ddtree_tree_attention_rope(q.float(), kc.float(), vc.float(), att.cu_prefix.tolist(), cu, kt.float(), vt.float(),
                                      mask, n_rows, pos, 1e6)
    assert e.value.status == 2
