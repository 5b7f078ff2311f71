"""GPU parity of ddtree_build and ddtree_accept against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import ddtree_oracle as orc
from paper_2604_12989_b200 import workloads as wl
from tests import ddtree_cases as cases

pytestmark = pytest.mark.gpu


def run_build(w, logits_np, roots_np, bf16_logits=False):
    import paper_2604_12989_b200 as dd
    x = torch.from_numpy(logits_np).cuda()
    if bf16_logits:
        x = x.to(torch.bfloat16)
    V = x.shape[-1]
    x = torch.nn.functional.pad(x, (0, (-V) % 8))[:, :, :V]  # rows start on 16-byte boundaries
    roots = torch.from_numpy(roots_np).cuda()
    plen = torch.tensor(w.prefix_lens, dtype=torch.int32).cuda()
    # outputs and workspace between poisoned guard bands: nothing may be written outside them
    g = cases.Guard()
    out = cases.guarded_tree(g, w.R, w.L, w.K, w.B)
    ws = g.empty((max(256, dd.lib().ddtree_build_workspace_bytes(w.R, w.L, V, w.K, w.B)),), torch.uint8)
    tree = dd.ddtree_build(x, w.K, w.B, roots, plen, workspace=ws, out=out)
    g.check()
    return tree


def check_build(w, variant):
    logits = cases.drafter_batch(w, variant)
    roots = wl.root_tokens(w)
    trees = cases.oracle_trees(w, logits, roots)
    tree = run_build(w, logits, roots)
    for r in range(w.R):
        cases.tree_arrays_equal(trees[r], tree, r)
        tok, lq = orc.top_k(logits[r], w.K)
        np.testing.assert_array_equal(tree.topk_token[r].cpu().numpy(), tok)
        np.testing.assert_allclose(tree.topk_logprob[r].cpu().numpy(), lq, atol=2e-5, rtol=0)
    return logits, roots, trees, tree


def check_accept(w, variant, trees, tree):
    import paper_2604_12989_b200 as dd
    tl = np.stack([wl.target_logits(w, trees[r].depth, r, variant) for r in range(w.R)])
    t = cases.to_torch(tl, w.dtype == "bf16")
    g = cases.Guard()
    ws = g.empty((max(256, dd.lib().ddtree_accept_workspace_bytes(w.R, w.B, w.V)),), torch.uint8)
    acc = dd.ddtree_accept(t, w.L, tree.node_token, tree.node_parent, tree.n_rows, workspace=ws,
                           out=cases.guarded_acceptance(g, w.R, w.L, w.N))
    g.check()
    lens = []
    for r in range(w.R):
        choice = orc.node_argmax(cases.to_f64(w, tl[r]))
        n = trees[r].n_rows
        want = orc.accept_walk(trees[r].token, trees[r].parent, n, choice)
        got_am = acc.node_argmax[r].cpu().numpy()
        np.testing.assert_array_equal(got_am[:n], choice[:n])
        assert (got_am[n:] == -1).all()
        assert int(acc.accept_len[r]) == want.accept_len
        nodes = acc.accept_nodes[r].cpu().numpy()
        toks = acc.accept_tokens[r].cpu().numpy()
        assert list(nodes[:want.accept_len]) == want.nodes and (nodes[want.accept_len:] == -1).all()
        assert list(toks[:want.accept_len]) == want.tokens and (toks[want.accept_len:] == -1).all()
        assert int(acc.bonus_token[r]) == want.bonus_token
        lens.append(want.accept_len)
    return lens


@pytest.mark.parametrize("variant", wl.VARIANTS)
@pytest.mark.parametrize("cfg", [0, 1, 2, 3, 4])
def test_build_and_accept_on_the_five_workloads(cfg, variant):
    w = wl.WORKLOADS[cfg]
    _, _, trees, tree = check_build(w, variant)
    lens = check_accept(w, variant, trees, tree)
    if variant == "peak":
        assert max(lens) >= 3  # the walk is actually exercised


def test_build_twice_is_bit_identical():
    w = wl.WORKLOADS[1]
    logits = cases.drafter_batch(w, "peak")
    roots = wl.root_tokens(w)
    a = run_build(w, logits, roots)
    b = run_build(w, logits, roots)
    for name in ("n_rows", "node_token", "node_parent", "node_depth", "position_ids", "anc_mask", "node_logprob",
                 "topk_token", "topk_logprob"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name


@pytest.mark.parametrize("R,L,V,K,B", [
    (1, 1, 8, 1, 1), (2, 3, 33, 2, 5), (3, 4, 1000, 4, 31), (2, 5, 1004, 5, 32), (1, 8, 5000, 1, 20),
    (2, 32, 4100, 32, 1024), (1, 16, 20000, 16, 1023), (4, 7, 777 * 4, 3, 200), (1, 2, 64, 32, 500),
    (2, 6, 12292, 8, 96), (1, 3, 4, 4, 84), (1, 3, 4, 4, 100),
])
def test_build_shapes_and_edges(R, L, V, K, B):
    """Odd vocabulary sizes (ragged 16-byte tail), K = 1, heaps that run empty, the maximum sizes,
    budgets around the 32-row mask-word boundary."""
    w = wl.small_workload(R=R, L=L, V=V, K=K, B=B, prefix_lens=tuple(range(3, 3 + R)), index=20)
    # every request is redrawn until its top-B set is unambiguous (boundary gap >= 1e-3); never skipped
    logits = cases.drafter_batch(w, "peak", seed=R * 1000 + V)
    roots = wl.root_tokens(w)
    trees = cases.oracle_trees(w, logits, roots)
    for r in range(R):
        _, lq = orc.top_k(logits[r], K)
        assert orc.boundary_gap(lq, B) >= 1e-3
    tree = run_build(w, logits, roots)
    for r in range(R):
        cases.tree_arrays_equal(trees[r], tree, r)


def test_build_bf16_logits_and_exact_ties():
    """bf16 logits tie exactly all over the vocabulary; ranks must still follow (value desc, id asc).
    K = 1 and B = L keep the tree a chain, so sigma ties between unrelated prefixes cannot matter."""
    w = wl.small_workload(R=2, L=6, V=6000, K=1, B=6, prefix_lens=(5, 9), index=21)
    rng = np.random.default_rng(5)
    x = wl.round_through_bf16(np.round(rng.standard_normal((2, 6, 6000)).astype(np.float32) * 4) / 4)
    roots = wl.root_tokens(w)
    trees = cases.oracle_trees(w, x, roots)
    for bf16 in (False, True):
        tree = run_build(w, x, roots, bf16_logits=bf16)
        for r in range(2):
            cases.tree_arrays_equal(trees[r], tree, r)


def test_topk_table_with_ties_wide_k():
    """Top-K membership and order under many exact ties, checked on the table output alone."""
    import paper_2604_12989_b200 as dd
    rng = np.random.default_rng(6)
    x = (np.round(rng.standard_normal((1, 4, 9001)).astype(np.float32) * 2) / 2)
    xt = torch.from_numpy(np.pad(x, ((0, 0), (0, 0), (0, 3)))).cuda()[:, :, :9001]  # row stride 9004: 16-byte rows
    tree = dd.ddtree_build(xt, 32, 8, torch.zeros(1, dtype=torch.int32).cuda(), torch.zeros(1, dtype=torch.int32).cuda())
    torch.cuda.synchronize()
    tok, lq = orc.top_k(x[0], 32)
    np.testing.assert_array_equal(tree.topk_token[0].cpu().numpy(), tok)
    np.testing.assert_allclose(tree.topk_logprob[0].cpu().numpy(), lq, atol=2e-5, rtol=0)


@pytest.mark.parametrize("want_len", [0, 1, 2, 5, 8])
def test_forced_acceptance_lengths(want_len):
    """Plant the target's choices along a chosen root path, preferring rank >= 2 children, and cut
    the path after `want_len` nodes; also covers argmax ties (lowest id wins)."""
    import paper_2604_12989_b200 as dd
    w = wl.small_workload(R=1, L=8, V=3000, K=4, B=60, index=22)
    logits = wl.drafter_logits(w, 0, "peak", seed=want_len)[None]
    roots = wl.root_tokens(w)
    ct = cases.oracle_trees(w, logits, roots)[0]
    tree = run_build(w, logits, roots)
    cases.tree_arrays_equal(ct, tree, 0)
    rng = np.random.default_rng(want_len)
    t = np.round(rng.standard_normal((w.N, w.V)).astype(np.float32) * 2) / 2  # lattice: ties at the top are common
    cur, path = 0, []
    while len(path) < want_len and ct.child_count[cur] > 0:
        kids = list(range(ct.first_child[cur], ct.first_child[cur] + ct.child_count[cur]))
        deeper = [k for k in kids if ct.child_count[k] > 0] or kids
        nxt = deeper[-1]  # highest rank that still has children
        t[cur, ct.token[nxt]] = 50.0
        path.append(nxt)
        cur = nxt
    # at the end of the path the target picks a token that is no child of `cur`; make it a tie
    kid_tokens = {int(ct.token[k]) for k in range(ct.n_rows) if ct.parent[k] == cur}
    free = [v for v in range(w.V) if v not in kid_tokens][:2]
    t[cur, free[0]] = 60.0
    t[cur, free[1]] = 60.0
    acc = dd.ddtree_accept(torch.from_numpy(t[None]).cuda(), w.L, tree.node_token, tree.node_parent, tree.n_rows)
    torch.cuda.synchronize()
    want = orc.accept_walk(ct.token, ct.parent, ct.n_rows, orc.node_argmax(t))
    assert want.accept_len == len(path) and want.bonus_token == min(free)
    assert int(acc.accept_len[0]) == want.accept_len
    assert list(acc.accept_nodes[0].cpu().numpy()[:want.accept_len]) == want.nodes
    assert int(acc.bonus_token[0]) == want.bonus_token
    np.testing.assert_array_equal(acc.node_argmax[0].cpu().numpy()[:ct.n_rows], orc.node_argmax(t)[:ct.n_rows])


def test_accept_full_depth_chain_and_bf16_ties():
    import paper_2604_12989_b200 as dd
    w = wl.small_workload(R=3, L=5, V=4099 + 5, K=1, B=9, prefix_lens=(1, 2, 3), index=23)  # heap runs empty: n_rows = 6 < 10
    logits = np.stack([wl.drafter_logits(w, r, "peak") for r in range(3)])
    roots = wl.root_tokens(w)
    trees = cases.oracle_trees(w, logits, roots)
    tree = run_build(w, logits, roots)
    rng = np.random.default_rng(1)
    t = np.round(rng.standard_normal((3, w.N, w.V)).astype(np.float32) * 2) / 2
    for r in range(3):
        cases.tree_arrays_equal(trees[r], tree, r)
        assert trees[r].n_rows == 6
        for i in range(5 if r < 2 else 3):  # request 2 stops after 3
            t[r, i, trees[r].token[i + 1]] = 40.0
    tb = wl.f32_to_bf16_bits(t)
    acc = dd.ddtree_accept(cases.to_torch(tb, True), w.L, tree.node_token, tree.node_parent, tree.n_rows)
    torch.cuda.synchronize()
    for r in range(3):
        want = orc.accept_walk(trees[r].token, trees[r].parent, 6, orc.node_argmax(wl.bf16_to_f64(tb[r])))
        assert int(acc.accept_len[r]) == want.accept_len == (5 if r < 2 else 3)
        assert int(acc.bonus_token[r]) == want.bonus_token
        assert list(acc.accept_nodes[r].cpu().numpy()[:want.accept_len]) == want.nodes


def test_argument_errors_launch_nothing():
    import paper_2604_12989_b200 as dd
    x = torch.zeros(1, 2, 64, device="cuda")
    z = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(dd.DDTreeError) as e:
        dd.ddtree_build(x, 65, 4, z, z)  # K > V
    assert e.value.status == 1
    with pytest.raises(dd.DDTreeError):
        dd.ddtree_build(x, 33, 4, z, z)  # K > 32
    with pytest.raises(dd.DDTreeError):
        dd.ddtree_build(x, 4, 1025, z, z)  # B > 1024
    with pytest.raises(dd.DDTreeError) as e:
        dd.ddtree_build(x, 4, 4, z, z, workspace=torch.zeros(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3
    with pytest.raises(dd.DDTreeError):
        dd.ddtree_build(x[:, :, 1:], 4, 4, z, z)  # rows not 16-byte aligned
    dd.device_status()


def test_build_full_vocab_bf16_logits_ragged_batch():
    """Drafter logits given as bf16 at full vocabulary size.  The retained logits of every position
    are placed on the bf16 lattice with irregular gaps (multiples of 0.25 below 64), so the input is
    exactly representable and the top-B set is still unambiguous."""
    w = wl.small_workload(R=3, L=16, V=151936, K=8, B=48, prefix_lens=(10, 20, 30), noise=3.0, boost0=8.0,
                          boost_slope=0.4, index=24)
    roots = wl.root_tokens(w)
    for attempt in range(200):
        rng = np.random.default_rng([24, attempt])
        xb = wl.round_through_bf16(np.stack([wl.drafter_logits(w, r, "lit", attempt) for r in range(3)]))
        for r in range(3):
            for i in range(w.L):
                top = np.argsort(-xb[r, i], kind="stable")[: w.K + 1]
                steps = rng.integers(1, 6, w.K + 1) * 0.25
                vals = 20.0 + np.cumsum(steps[::-1])[::-1]  # strictly decreasing, all multiples of 0.25 in (20, 30)
                xb[r, i, top] = vals.astype(np.float32)
        assert np.array_equal(wl.round_through_bf16(xb), xb)
        ok = all(orc.boundary_gap(orc.top_k(xb[r], w.K)[1], w.B) >= 1e-3 for r in range(3))
        if ok:
            break
    else:
        pytest.fail("no draw with an unambiguous top-B set in 200 attempts")
    trees = cases.oracle_trees(w, xb, roots)
    tree = run_build(w, xb, roots, bf16_logits=True)
    for r in range(3):
        cases.tree_arrays_equal(trees[r], tree, r)
        assert trees[r].depth.max() >= 2


def test_accept_ragged_vocab_tail_bf16():
    """V = 5003 in bf16: rows are padded to 16-byte starts, the last 3 elements are read one by one."""
    import paper_2604_12989_b200 as dd
    w = wl.small_workload(R=2, L=5, V=5003, K=3, B=25, prefix_lens=(1, 2), dtype="bf16", index=25)
    logits = np.stack([wl.drafter_logits(w, r, "peak") for r in range(2)])
    roots = wl.root_tokens(w)
    trees = cases.oracle_trees(w, logits, roots)
    tree = run_build(w, logits, roots)
    tl = np.stack([wl.target_logits(w, trees[r].depth, r, "peak") for r in range(2)])
    for r in range(2):  # put the maximum of some rows into the ragged tail
        tl[r, 0, 5002] = wl.f32_to_bf16_bits(np.array([80.0], np.float32))[0]
        tl[r, 1, 5000] = wl.f32_to_bf16_bits(np.array([90.0], np.float32))[0]
    t = cases.to_torch(tl, True)
    t = torch.nn.functional.pad(t, (0, 5))[:, :, :5003]
    acc = dd.ddtree_accept(t, w.L, tree.node_token, tree.node_parent, tree.n_rows)
    torch.cuda.synchronize()
    for r in range(2):
        choice = orc.node_argmax(wl.bf16_to_f64(tl[r]))
        assert choice[0] == 5002 and choice[1] == 5000
        n = trees[r].n_rows
        np.testing.assert_array_equal(acc.node_argmax[r].cpu().numpy()[:n], choice[:n])
        want = orc.accept_walk(trees[r].token, trees[r].parent, n, choice)
        assert int(acc.accept_len[r]) == want.accept_len and int(acc.bonus_token[r]) == want.bonus_token
