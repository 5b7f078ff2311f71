"""ddtree_accept_static_scratch: the variant of ddtree_accept for callers that cannot obtain device
memory for a workspace (a decoding loop whose memory pool is fully committed, a plug-in without an
allocator).  Its scratch is a fixed array inside the library, so the test checks, through the C
ABI, that two calls in a row give exactly what ddtree_accept gives with a caller workspace (and what
the CPU oracle's walk gives), that the call leaves torch's allocator untouched, and that a problem too
large for the array is refused.  Collected last on purpose: if it fails, a run that stops at the first
failure has already run every other test."""
import numpy as np
import pytest
import torch

from oracle import ddtree_oracle as orc
from paper_2604_12989_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def make_round(seed, w):
    import paper_2604_12989_b200 as dd
    logits = torch.from_numpy(np.stack([wl.drafter_logits(w, r, "peak", seed) for r in range(w.R)])).cuda()
    roots = torch.from_numpy(wl.root_tokens(w, seed)).cuda()
    plen = torch.tensor(w.prefix_lens, dtype=torch.int32).cuda()
    tree = dd.ddtree_build(logits, w.K, w.B, roots, plen)
    torch.cuda.synchronize()
    depth = tree.node_depth.cpu().numpy()
    target = np.stack([wl.target_logits(w, depth[r], r, "peak", seed) for r in range(w.R)])
    return tree, torch.from_numpy(target).cuda(), target


def empty_acceptance(w):
    import paper_2604_12989_b200 as dd
    i32 = dict(dtype=torch.int32, device="cuda")
    return dd.Acceptance(torch.full((w.R,), -7, **i32), torch.full((w.R, w.L), -7, **i32),
                         torch.full((w.R, w.L), -7, **i32), torch.full((w.R,), -7, **i32),
                         torch.full((w.R, w.N), -7, **i32))


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    import paper_2604_12989_b200 as dd
    w = wl.small_workload(R=3, L=8, V=20000, K=4, B=40, prefix_lens=(5, 6, 7), index=60)
    assert dd.lib().ddtree_accept_workspace_bytes(w.R, w.B, w.V) <= dd.STATIC_SCRATCH_BYTES
    for seed in (0, 1):  # two calls in a row: the second one meets the first one's leftovers in the array
        tree, target, target_h = make_round(seed, w)
        want = dd.ddtree_accept(target, w.L, tree.node_token, tree.node_parent, tree.n_rows)
        out = empty_acceptance(w)
        torch.cuda.synchronize()
        counters = lambda: (torch.cuda.memory_stats()["allocation.all.allocated"], torch.cuda.memory_reserved())
        before = counters()  # allocation requests served so far, bytes held from the driver
        got = dd.ddtree_accept_static_scratch(target, w.L, tree.node_token, tree.node_parent, tree.n_rows, out=out)
        torch.cuda.synchronize()
        assert counters() == before  # the call asked torch's allocator for nothing, and nothing was reserved
        for name in ("accept_len", "accept_nodes", "accept_tokens", "bonus_token", "node_argmax"):
            assert torch.equal(getattr(got, name), getattr(want, name)), (seed, name)
        assert int(want.accept_len.max()) >= 1  # the walk did something
        # and the CPU oracle agrees: the target's greedy choice at every row, the walk over them
        tok, par, n_rows = tree.node_token.cpu().numpy(), tree.node_parent.cpu().numpy(), tree.n_rows.cpu().numpy()
        for r in range(w.R):
            n = int(n_rows[r])
            choice = orc.node_argmax(target_h[r].astype(np.float64))
            np.testing.assert_array_equal(got.node_argmax[r].cpu().numpy()[:n], choice[:n])
            walk = orc.accept_walk(tok[r], par[r], n, choice)
            assert int(got.accept_len[r]) == walk.accept_len and int(got.bonus_token[r]) == walk.bonus_token
            assert list(got.accept_nodes[r].cpu().numpy()[:walk.accept_len]) == walk.nodes


def test_static_scratch_refuses_what_does_not_fit():
    import paper_2604_12989_b200 as dd
    w = wl.small_workload(R=40, L=4, V=151936, K=2, B=1024, prefix_lens=tuple([1] * 40), index=61)
    assert dd.lib().ddtree_accept_workspace_bytes(w.R, w.B, w.V) > dd.STATIC_SCRATCH_BYTES
    t = torch.zeros(1, 2, 8, device="cuda")  # never read: the size check comes first
    z = torch.zeros(w.R, w.N, dtype=torch.int32, device="cuda")
    rc = dd.lib().ddtree_accept_static_scratch(t.data_ptr(), 0, 8, w.R, w.B, w.V, w.L, z.data_ptr(), z.data_ptr(),
                                               z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(),
                                               None, None)
    assert rc == 3
    assert b"built-in array" in dd.lib().ddtree_last_error()
