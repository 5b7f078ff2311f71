"""GPU parity of ddtree_tree_attention against the fp64 CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import ddtree_oracle as orc
from paper_2604_12989_b200 import workloads as wl
from tests import ddtree_cases as cases

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 1e-2}


def gpu_attention(w, att, trees, with_lse=True):
    import paper_2604_12989_b200 as dd
    bf = w.dtype == "bf16"
    mask = torch.from_numpy(np.stack([t.mask for t in trees]).view(np.int32)).cuda()
    n_rows = torch.tensor([t.n_rows for t in trees], dtype=torch.int32).cuda()
    cu = torch.from_numpy(att.cu_prefix).cuda()
    q, kc, vc, kt, vt = (cases.to_torch(getattr(att, n), bf) for n in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
    lse = torch.zeros(w.R, w.N, w.Hq, dtype=torch.float32, device="cuda") if with_lse else None
    out = dd.ddtree_tree_attention(q, kc, vc, att.cu_prefix.tolist(), cu, kt, vt, mask, n_rows, lse=lse)
    torch.cuda.synchronize()
    dd.device_status()
    return out.float().cpu().numpy().astype(np.float64), (lse.cpu().numpy() if with_lse else None)


def compare(w, att, trees, out, lse, rows_heads=None):
    """Element-wise |gpu - oracle| <= tol * (1 + |oracle|) on all rows (or on sampled (row, head) pairs)."""
    tol = TOL[w.dtype]
    worst = 0.0
    for r in range(w.R):
        lo, hi = att.cu_prefix[r], att.cu_prefix[r + 1]
        args = (att.as_f64("q")[r], att.as_f64("k_cache")[lo:hi], att.as_f64("v_cache")[lo:hi],
                att.as_f64("k_tree")[r], att.as_f64("v_tree")[r], trees[r].mask, trees[r].n_rows)
        if rows_heads is None:
            ref, ref_lse = orc.tree_attention(*args)
            got = out[r, :trees[r].n_rows]
            err = np.abs(got - ref) / (1 + np.abs(ref))
            worst = max(worst, err.max())
            assert err.max() <= tol, f"request {r}: max scaled error {err.max():.3e}"
            if lse is not None:
                np.testing.assert_allclose(lse[r, :trees[r].n_rows], ref_lse, atol=tol, rtol=tol)
        else:
            for (i, h) in rows_heads[r]:
                ref, ref_lse = orc.tree_attention(*args, rows=[i], heads=[h])
                err = np.abs(out[r, i, h] - ref[0, 0]) / (1 + np.abs(ref[0, 0]))
                worst = max(worst, err.max())
                assert err.max() <= tol, f"request {r} row {i} head {h}: {err.max():.3e}"
                if lse is not None:
                    assert abs(lse[r, i, h] - ref_lse[0, 0]) <= tol * (1 + abs(ref_lse[0, 0]))
    return worst


def make_case(w, variant="peak", seed=0):
    logits = np.stack([wl.drafter_logits(w, r, variant, seed) for r in range(w.R)])
    trees = cases.oracle_trees(w, logits, wl.root_tokens(w, seed))
    att = wl.attention_inputs(w, 0, seed)
    return att, trees


def test_config0_fp32():
    w = wl.WORKLOADS[0]
    for variant in wl.VARIANTS:
        att, trees = make_case(w, variant)
        out, lse = gpu_attention(w, att, trees)
        compare(w, att, trees, out, lse)


@pytest.mark.parametrize("P", [0, 1, 7, 127, 129])
@pytest.mark.parametrize("d", [64, 128])
def test_fp32_short_prefixes_and_sentinel_values(P, d):
    """Short prefixes expose a wrong mask bit; tree V rows carry a large one-hot so that any leaked
    tree key breaks the tolerance.  Two requests, the second with a heap that ran empty."""
    w = wl.small_workload(R=2, L=6, V=500, K=3, B=70, Hq=4, Hkv=2, d=d, prefix_lens=(P, P + 5), index=30)
    att, trees = make_case(w)
    for r in range(2):
        for j in range(w.N):
            att.v_tree[r, j, :, :] = 0
            att.v_tree[r, j, :, j % d] = 1e4
    out, lse = gpu_attention(w, att, trees)
    compare(w, att, trees, out, lse)


def test_fp32_padding_rows_untouched_and_no_lse():
    w = wl.small_workload(R=1, L=4, V=300, K=1, B=9, Hq=2, Hkv=1, d=64, prefix_lens=(33,), index=31)
    att, trees = make_case(w)
    assert trees[0].n_rows == 5
    out, _ = gpu_attention(w, att, trees, with_lse=False)
    compare(w, att, trees, out, None)
    assert (out[0, 5:] == 0).all()
