"""GPU parity of ddtree_tree_attention against the fp64 CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import ddtree_oracle as orc
from paper_2604_12989_b200 import workloads as wl
from tests import ddtree_cases as cases

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 1e-2}


@pytest.fixture(params=["two_row_tiles", "one_row_tile"])
def kernel_path(request):
    """The library has two bf16 kernels and normally picks one per call from the shapes; tests that take this
    fixture run once with each forced (a forced choice that does not apply to a shape falls back to the other)."""
    import paper_2604_12989_b200 as dd
    dd.tree_attention_set_path(1 if request.param == "two_row_tiles" else 2)
    yield request.param
    dd.tree_attention_set_path(0)


def gpu_attention(w, att, trees, with_lse=True):
    import paper_2604_12989_b200 as dd
    bf = w.dtype == "bf16"
    mask = torch.from_numpy(np.stack([t.mask for t in trees]).view(np.int32)).cuda()
    n_rows = torch.tensor([t.n_rows for t in trees], dtype=torch.int32).cuda()
    cu = torch.from_numpy(att.cu_prefix).cuda()
    q, kc, vc, kt, vt = (cases.to_torch(getattr(att, n), bf) for n in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
    # out, lse and the workspace sit between poisoned guard bands: nothing may be written outside them
    g = cases.Guard()
    lse = g.empty((w.R, w.N, w.Hq), torch.float32, fill=0) if with_lse else None
    out = g.empty(tuple(q.shape), q.dtype, fill=0)
    ws = g.empty((max(256, dd.tree_attention_workspace_bytes(w.R, w.B, w.Hq, w.Hkv, w.d, 1 if bf else 0,
                                                             att.cu_prefix.tolist())),), torch.uint8)
    dd.ddtree_tree_attention(q, kc, vc, att.cu_prefix.tolist(), cu, kt, vt, mask, n_rows, out=out, lse=lse, workspace=ws)
    g.check()
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


# ---------------------------------------------------------------------------------------------
# bf16 (tensor-core path)
# ---------------------------------------------------------------------------------------------

def bf16_case(R, B, Hq, Hkv, prefix_lens, K=4, L=8, seed=0, sentinel=False):
    w = wl.small_workload(R=R, L=L, V=600, K=K, B=B, Hq=Hq, Hkv=Hkv, d=128, dtype="bf16",
                          prefix_lens=prefix_lens, index=40)
    att, trees = make_case(w, seed=seed)
    if sentinel:
        v = np.zeros((R, w.N, Hkv, 128), np.float32)
        for j in range(w.N):
            v[:, j, :, j % 128] = 1e3
        att.v_tree = wl.f32_to_bf16_bits(v)
    return w, att, trees


@pytest.mark.parametrize("P", [0, 1, 7, 127, 128, 129, 300])
def test_bf16_short_prefixes_and_sentinel_values(P, kernel_path):
    w, att, trees = bf16_case(2, 70, 8, 2, (P, P + 5 if P else 0), sentinel=True)
    out, lse = gpu_attention(w, att, trees)
    compare(w, att, trees, out, lse)


@pytest.mark.parametrize("profile", ["growing", "exploding", "shrinking"])
def test_bf16_scores_that_outgrow_the_reference_maximum(profile, kernel_path):
    # The kernel exponentiates a tile against the reference maximum it already has and looks at the
    # exact maximum only when a row sum comes near overflow.  Keys whose scale changes from one
    # 128-key tile to the next force that path: "growing" lifts the scores by ~2^30 per tile (row
    # sums pass 2^24), "exploding" by more than 2^128 (the optimistic exponentials are infinite),
    # "shrinking" puts the largest scores first (reference far above everything that follows).
    w, att, trees = bf16_case(1, 40, 8, 2, (6 * 128 + 17,), seed=11)
    k = wl.bf16_to_f64(att.k_cache).astype(np.float32)
    tiles = np.arange(k.shape[0]) // 128
    factor = {"growing": 1.0 + 6.0 * tiles, "exploding": 1.0 + 40.0 * tiles, "shrinking": 40.0 / (1.0 + 6.0 * tiles)}[profile]
    att.k_cache = wl.f32_to_bf16_bits(k * factor[:, None, None].astype(np.float32))
    out, lse = gpu_attention(w, att, trees)
    compare(w, att, trees, out, lse)


@pytest.mark.parametrize("G,Hkv", [(1, 2), (2, 2), (4, 1), (8, 1), (16, 1)])
def test_bf16_group_sizes(G, Hkv, kernel_path):
    w, att, trees = bf16_case(1, 40, G * Hkv, Hkv, (200,), seed=G)
    out, lse = gpu_attention(w, att, trees)
    compare(w, att, trees, out, lse)


def test_bf16_two_tree_tiles_and_heap_that_ran_empty(kernel_path):
    # B = 200: tree keys span two 128-key tiles; second request has K = 1 chain (n_rows = 9 << B+1)
    w, att, trees = bf16_case(2, 200, 4, 1, (260, 3), K=4, L=8, seed=3)
    chain = orc.build(wl.drafter_logits(w, 1, "peak", 3), 1, w.B, 0, 3)
    trees[1] = chain
    assert chain.n_rows == 9
    out, lse = gpu_attention(w, att, trees)
    compare(w, att, trees, out, lse)
    assert (out[1, 9:] == 0).all()  # padding rows untouched


# A last row tile of at most 16 rows (the root's G rows left over by a tree of 2^k nodes, typically)
# takes a path of its own when the batch fills the SMs several times over (R * Hkv * row tiles >= 148):
# keys on the TMEM lanes, swapped products, two groups of key threads taking alternate tiles.
# (R, B, Hq, Hkv): rows of the short tile = (B + 1) * G mod 128.
SHORT_TILE_SHAPES = [
    (38, 32, 8, 2),    # 4 rows
    (50, 64, 4, 1),    # 4 rows after two full tiles
    (40, 3, 16, 4),    # the whole problem is one short tile (16 rows) per KV head
    (150, 1, 8, 1),    # 2 nodes x 8 heads
    (75, 16, 8, 1),    # 8 rows
    (75, 8, 16, 1),    # 16 rows of one node
    (75, 35, 4, 1),    # 16 rows from 4 nodes
    (15, 128, 8, 2),   # two tree tiles
]


def short_tile_prefixes(R, seed, hi=400):
    p = [int(x) for x in np.random.default_rng(seed).integers(0, hi, R)]
    p[:5] = [0, 128, 129, 1, 2 * 128 + 7][:R]  # no prefix (tree keys only: one tile, one key group idle), tile boundaries
    return tuple(p)


@pytest.mark.parametrize("R,B,Hq,Hkv", SHORT_TILE_SHAPES)
def test_bf16_short_last_row_tile(R, B, Hq, Hkv):
    w, att, trees = bf16_case(R, B, Hq, Hkv, short_tile_prefixes(R, B), K=4, L=8, seed=B, sentinel=True)
    out, lse = gpu_attention(w, att, trees)
    compare(w, att, trees, out, lse)


def test_bf16_short_last_row_tile_partly_and_wholly_padding():
    # B = 35, G = 4: nodes 32..35 sit in the short tile.  Trees of 34, 9 and 36 rows: half of the short
    # tile, none of it, all of it.
    import dataclasses
    R = 75
    w, att, trees = bf16_case(R, 35, 4, 1, short_tile_prefixes(R, 7, 300), K=4, L=8, seed=2)
    assert all(t.n_rows == 36 for t in trees)
    for r in range(0, R, 3):
        trees[r] = dataclasses.replace(trees[r], n_rows=34)  # the first rows of a level-order tree are a tree
    for r in range(1, R, 3):
        trees[r] = orc.build(wl.drafter_logits(w, r, "peak", 2), 1, w.B, 0, 3)
        assert trees[r].n_rows == 9
    out, lse = gpu_attention(w, att, trees)
    compare(w, att, trees, out, lse)
    assert (out[0, 34:] == 0).all() and (out[1, 9:] == 0).all()


@pytest.mark.parametrize("profile", ["growing", "exploding", "shrinking"])
@pytest.mark.parametrize("R,B,prefix", [(19, 32, 6 * 128 + 17), (37, 3, 9 * 128 + 1)])
def test_bf16_short_last_row_tile_scores_that_outgrow_the_reference_maximum(profile, R, B, prefix):
    # as the test of that name for the full tiles: here the reference maximum is shared by the 128 key
    # threads of a group and the accumulated O^T has to be rescaled when it moves
    w, att, trees = bf16_case(R, B, 16, 4, (prefix,) * R, seed=13)
    k = wl.bf16_to_f64(att.k_cache).astype(np.float32)
    tiles = (np.arange(k.shape[0]) % prefix) // 128
    factor = {"growing": 1.0 + 6.0 * tiles, "exploding": 1.0 + 40.0 * tiles, "shrinking": 40.0 / (1.0 + 6.0 * tiles)}[profile]
    att.k_cache = wl.f32_to_bf16_bits(k * factor[:, None, None].astype(np.float32))
    out, lse = gpu_attention(w, att, trees)
    compare(w, att, trees, out, lse, rows_heads=[[(i, h) for i in range(trees[r].n_rows) for h in ((r % 16), 15 - (r % 16))] for r in range(R)])


def test_bf16_many_requests_direct_path_and_repeatability():
    # R * Hkv * row_tiles >= number of SMs: no KV split, outputs written directly
    prefix = tuple(int(x) for x in np.random.default_rng(1).integers(1, 400, 40))
    w, att, trees = bf16_case(40, 31, 16, 4, prefix, seed=5)
    out, lse = gpu_attention(w, att, trees)
    compare(w, att, trees, out, lse)
    out2, lse2 = gpu_attention(w, att, trees)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def sampled_pairs(w, trees, heads_full, n_random, seed):
    rng = np.random.default_rng(seed)
    out = []
    for r in range(w.R):
        n = trees[r].n_rows
        pairs = [(i, h) for h in heads_full for i in range(n)]
        pairs += [(int(rng.integers(0, n)), int(rng.integers(0, w.Hq))) for _ in range(n_random)]
        out.append(pairs)
    return out


@pytest.mark.parametrize("cfg,heads_full,n_random", [(1, tuple(range(32)), 0), (2, (0, 13), 32), (3, (5,), 16),
                                                      (4, (63,), 48)])
def test_bf16_full_size_workloads(cfg, heads_full, n_random):
    """The five workloads at full size in the launch configuration the benchmark times; the oracle
    evaluates all rows of the named heads plus random (row, head) pairs."""
    w = wl.WORKLOADS[cfg]
    att, trees = make_case(w, "peak")
    out, lse = gpu_attention(w, att, trees)
    worst = compare(w, att, trees, out, lse, sampled_pairs(w, trees, heads_full, n_random, cfg))
    print(f"config {cfg}: worst scaled error {worst:.3e}")


@pytest.mark.parametrize("cfg", [1, 2])
def test_bf16_full_size_one_request_on_either_kernel(cfg, kernel_path):
    """Workloads 1 and 2 (one request: every CTA resident at once, the KV range split) on each of the two kernels."""
    w = wl.WORKLOADS[cfg]
    att, trees = make_case(w, "peak", seed=3)
    out, lse = gpu_attention(w, att, trees)
    compare(w, att, trees, out, lse, sampled_pairs(w, trees, (7,), 24, 10 + cfg))


def test_bf16_first_call_of_a_fresh_process():
    """The first launch of a process runs with cold instruction caches and unusual warp timing; a
    missed wait inside the kernel shows up there first.  Two-tile, unsplit case in a child process."""
    import subprocess
    import sys
    code = (
        "import numpy as np\n"
        "from tests import test_gpu_attention as T\n"
        "w, att, trees = T.bf16_case(1, 20, 4, 1, (128,))\n"
        "out, lse = T.gpu_attention(w, att, trees)\n"
        "T.compare(w, att, trees, out, lse)\n"
        "print('fresh-process ok')\n")
    import os
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, "-c", code], cwd=root, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0 and "fresh-process ok" in res.stdout, res.stdout + res.stderr


def test_bf16_largest_tree_and_custom_scale(kernel_path):
    """B = 1024 (1025 rows, 33 mask words, nine 128-key tree tiles), empty prefix, 16 query heads per KV
    head, a caller-chosen softmax scale and no lse output."""
    import paper_2604_12989_b200 as dd
    w = wl.small_workload(R=1, L=12, V=3000, K=6, B=1024, Hq=16, Hkv=1, d=128, dtype="bf16", prefix_lens=(0,), index=41)
    att, trees = make_case(w)
    assert trees[0].n_rows == 1025
    mask = torch.from_numpy(trees[0].mask[None].view(np.int32)).cuda()
    n_rows = torch.tensor([1025], dtype=torch.int32).cuda()
    cu = torch.from_numpy(att.cu_prefix).cuda()
    q, kc, vc, kt, vt = (cases.to_torch(getattr(att, n), True) for n in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
    kc = torch.zeros(1, 1, 128, dtype=torch.bfloat16, device="cuda")  # empty prefix: never read
    vc = torch.zeros_like(kc)
    out = dd.ddtree_tree_attention(q, kc, vc, [0, 0], cu, kt, vt, mask, n_rows, softmax_scale=0.05)
    torch.cuda.synchronize()
    dd.device_status()
    got = out.float().cpu().numpy().astype(np.float64)
    rng = np.random.default_rng(0)
    empty = np.zeros((0, 1, 128))
    for _ in range(40):
        i, h = int(rng.integers(0, 1025)), int(rng.integers(0, 16))
        ref, _ = orc.tree_attention(att.as_f64("q")[0], empty, empty, att.as_f64("k_tree")[0], att.as_f64("v_tree")[0],
                                    trees[0].mask, 1025, scale=0.05, rows=[i], heads=[h])
        err = np.abs(got[0, i, h] - ref[0, 0]) / (1 + np.abs(ref[0, 0]))
        assert err.max() <= 1e-2, (i, h, err.max())


def test_bf16_batch_with_an_empty_prefix_and_a_root_only_tree(kernel_path):
    """Request 0 has no cached context, request 2's tree is the root alone (n_rows = 1)."""
    w = wl.small_workload(R=3, L=6, V=900, K=3, B=37, Hq=8, Hkv=2, d=128, dtype="bf16", prefix_lens=(0, 700, 130), index=42)
    att, trees = make_case(w)
    root_only = orc.compile_tree([], np.zeros((6, 3), np.int64), 5, 130, w.B)
    assert root_only.n_rows == 1
    trees[2] = root_only
    out, lse = gpu_attention(w, att, trees)
    compare(w, att, trees, out, lse)
    assert (out[2, 1:] == 0).all()


def test_bf16_workspace_too_small_is_refused():
    import paper_2604_12989_b200 as dd
    w, att, trees = bf16_case(1, 64, 8, 2, (2000,))
    mask = torch.from_numpy(np.stack([t.mask for t in trees]).view(np.int32)).cuda()
    n_rows = torch.tensor([t.n_rows for t in trees], dtype=torch.int32).cuda()
    q, kc, vc, kt, vt = (cases.to_torch(getattr(att, n), True) for n in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
    need = dd.tree_attention_workspace_bytes(1, 64, 8, 2, 128, 1, att.cu_prefix.tolist())
    assert need > 4096
    with pytest.raises(dd.DDTreeError) as e:
        dd.ddtree_tree_attention(q, kc, vc, att.cu_prefix.tolist(), torch.from_numpy(att.cu_prefix).cuda(), kt, vt, mask,
                                 n_rows, workspace=torch.zeros(4096, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3
    with pytest.raises(dd.DDTreeError) as e:  # head_dim 64 has no bf16 kernel
        dd.ddtree_tree_attention(q[..., :64].contiguous(), kc[..., :64].contiguous(), vc[..., :64].contiguous(),
                                 att.cu_prefix.tolist(), torch.from_numpy(att.cu_prefix).cuda(),
                                 kt[..., :64].contiguous(), vt[..., :64].contiguous(), mask, n_rows)
    assert e.value.status == 2


@pytest.mark.parametrize("seed", range(14))
def test_bf16_random_shapes(seed, kernel_path):
    """Random small problems: batch size, budget, group size, prefix lengths (zero, a few keys, ragged
    ends of a 128-key tile, several tiles so that the KV range is split) and trees smaller than the
    budget, all rows against the oracle."""
    rng = np.random.default_rng(1000 + seed)
    R = int(rng.integers(1, 5))
    G = int(rng.choice([1, 2, 4, 8, 16]))
    Hkv = int(rng.choice([1, 2])) if G >= 8 else int(rng.choice([1, 2, 4]))
    B = int(rng.choice([1, 2, 7, 31, 32, 33, 63, 64, 100, 129, 200, 300]))
    kinds = [0, int(rng.integers(1, 8)), 127, 128, 129, int(rng.integers(130, 700)), int(rng.integers(700, 2600))]
    prefix = tuple(int(rng.choice(kinds)) for _ in range(R))
    L = int(rng.integers(2, 9))
    K = int(rng.integers(1, 5))
    w, att, trees = bf16_case(R, B, G * Hkv, Hkv, prefix, K=K, L=L, seed=seed)
    out, lse = gpu_attention(w, att, trees)
    compare(w, att, trees, out, lse)
    for r in range(R):
        assert (out[r, trees[r].n_rows:] == 0).all()  # rows past the tree are left alone


def test_bf16_padding_inputs_may_hold_nan(kernel_path):
    """Rows of the inputs that the call must ignore are filled with NaN bit patterns: tree rows >= n_rows of
    q, k_tree and v_tree (one request's tree is smaller than the budget), and spare cache rows behind the
    last request's prefix.  Masked probabilities are zero, but the value rows of a masked key still travel
    through the tensor cores in a 128-key tile, so the kernel has to clear them: every valid row must still
    match the oracle, on the split path (one request), on the unsplit path (a batch that fills the GPU) and
    on the short last row tile."""
    import dataclasses
    import paper_2604_12989_b200 as dd
    nan16 = np.uint16(0x7FC0)
    for R, B, Hq, Hkv, prefix in ((1, 200, 8, 2, (300,)), (2, 70, 8, 2, (127, 5)), (40, 35, 16, 4, None), (75, 35, 4, 1, None)):
        if prefix is None:
            prefix = short_tile_prefixes(R, B, 300)
        w, att, trees = bf16_case(R, B, Hq, Hkv, prefix, seed=B)
        for r in range(0, R, 2):  # every other request: a smaller tree (the first rows of a level-order tree are a tree)
            trees[r] = dataclasses.replace(trees[r], n_rows=max(1, trees[r].n_rows - 3 - r % 5))
        for r in range(R):
            n = trees[r].n_rows
            att.q[r, n:] = nan16
            att.k_tree[r, n:] = nan16
            att.v_tree[r, n:] = nan16
        bf = True
        mask = torch.from_numpy(np.stack([t.mask for t in trees]).view(np.int32)).cuda()
        n_rows = torch.tensor([t.n_rows for t in trees], dtype=torch.int32).cuda()
        cu = torch.from_numpy(att.cu_prefix).cuda()
        q, kc, vc, kt, vt = (cases.to_torch(getattr(att, nm), bf) for nm in ("q", "k_cache", "v_cache", "k_tree", "v_tree"))
        # spare rows behind the packed cache (what a cache with room for the accepted path looks like)
        spare = torch.full((64,) + tuple(kc.shape[1:]), float("nan"), dtype=kc.dtype, device="cuda")
        kc2, vc2 = torch.cat([kc, spare]), torch.cat([vc, spare])
        total = int(att.cu_prefix[-1])
        out = torch.zeros_like(q)
        lse = torch.zeros(w.R, w.N, w.Hq, dtype=torch.float32, device="cuda")
        dd.ddtree_tree_attention(q, kc2[:total], vc2[:total], att.cu_prefix.tolist(), cu, kt, vt, mask, n_rows, out=out, lse=lse)
        torch.cuda.synchronize()
        dd.device_status()
        got = out.float().cpu().numpy().astype(np.float64)
        for r in range(R):  # the oracle never looks at rows >= n_rows
            n = trees[r].n_rows
            assert np.isfinite(got[r, :n]).all(), f"request {r}: NaN leaked into a valid row"
            assert (got[r, n:] == 0).all()
        compare(w, att, trees, got, lse.cpu().numpy())


def test_bf16_long_trains_of_launches_stay_identical(kernel_path):
    """Hundreds of back-to-back launches on the large-budget workload's shapes, rotating over input sets larger
    than L2 so that the copies' arrival order varies: every launch must give bit for bit what the first launch
    on the same inputs gave, and no device-side wait may give up.  (A warp that watched only every other phase
    of a copy barrier once passed a wait early when a K tile landed after the V tile behind it: a rare
    timing, seen only in long trains.)"""
    import paper_2604_12989_b200 as dd
    w = wl.WORKLOADS[2]
    att, trees = make_case(w, "lit")
    mask = torch.from_numpy(np.stack([t.mask for t in trees]).view(np.int32)).cuda()
    n_rows = torch.tensor([t.n_rows for t in trees], dtype=torch.int32).cuda()
    cu = torch.from_numpy(att.cu_prefix).cuda()
    base = [cases.to_torch(getattr(att, n), True) for n in ("q", "k_cache", "v_cache", "k_tree", "v_tree")]
    sets = [base] + [[torch.randn_like(t, dtype=torch.float32).to(torch.bfloat16) for t in base] for _ in range(2)]
    ws = torch.empty(max(256, dd.tree_attention_workspace_bytes(w.R, w.B, w.Hq, w.Hkv, w.d, 1, att.cu_prefix.tolist())),
                     dtype=torch.uint8, device="cuda")
    outs = [torch.zeros_like(base[0]) for _ in sets]
    first = []
    for k, (q, kc, vc, kt, vt) in enumerate(sets):
        dd.ddtree_tree_attention(q, kc, vc, att.cu_prefix.tolist(), cu, kt, vt, mask, n_rows, out=outs[k], workspace=ws)
        first.append(outs[k].clone())
    torch.cuda.synchronize()
    dd.device_status()
    for it in range(600):
        k = it % len(sets)
        q, kc, vc, kt, vt = sets[k]
        dd.ddtree_tree_attention(q, kc, vc, att.cu_prefix.tolist(), cu, kt, vt, mask, n_rows, out=outs[k], workspace=ws)
        if it % 100 == 99:
            torch.cuda.synchronize()
            for a, b in zip(outs, first):
                assert torch.equal(a, b), f"launch {it}: output changed"
    torch.cuda.synchronize()
    dd.device_status()
    out0 = first[0].float().cpu().numpy().astype(np.float64)
    compare(w, att, trees, out0, None, sampled_pairs(w, trees, (), 24, 2))
