"""GPU parity of ddtree_accept_sampled (Section 4.4, temperature-based decoding rule) against the CPU
oracle, through the C ABI: the drawn token of every row and the walk are compared bit for bit."""
import numpy as np
import pytest
import torch

from oracle import ddtree_oracle as orc
from paper_2604_12989_b200 import workloads as wl
from tests import ddtree_cases as cases

pytestmark = pytest.mark.gpu


def f32_rows(w, tl):
    """The logits the kernel sees, as float32 (bf16 bit patterns widen exactly)."""
    return wl.bf16_to_f64(tl).astype(np.float32) if w.dtype == "bf16" else tl.astype(np.float32)


def aligned_rows(t):
    """Same values, rows starting on 16-byte boundaries (odd vocabulary sizes)."""
    V = t.shape[-1]
    return torch.nn.functional.pad(t, (0, (-V) % 8))[..., :V]


def run_and_compare(w, trees, tl, T, ks):
    """tl: [R, N, V] (float32, or bf16 bits); ks: [R, N] uint32."""
    import paper_2604_12989_b200 as dd
    t = aligned_rows(cases.to_torch(tl, w.dtype == "bf16"))
    tok = torch.from_numpy(np.stack([tr.token for tr in trees])).cuda()
    par = torch.from_numpy(np.stack([tr.parent for tr in trees])).cuda()
    n_rows = torch.tensor([tr.n_rows for tr in trees], dtype=torch.int32).cuda()
    u = torch.from_numpy(ks.astype(np.uint32).view(np.int32)).cuda()
    g = cases.Guard()
    ws = g.empty((max(256, dd.lib().ddtree_accept_sampled_workspace_bytes(w.R, w.B, w.V)),), torch.uint8)
    acc = dd.ddtree_accept_sampled(t, w.L, tok, par, n_rows, T, u, workspace=ws,
                                   out=cases.guarded_acceptance(g, w.R, w.L, w.N))
    g.check()
    lens = []
    for r in range(w.R):
        n = trees[r].n_rows
        x = f32_rows(w, tl[r])
        choice = orc.node_sampled(x[:n], T, ks[r, :n])
        got = acc.node_argmax[r].cpu().numpy()
        np.testing.assert_array_equal(got[:n], choice)
        assert (got[n:] == -1).all()
        want = orc.accept_walk(trees[r].token, trees[r].parent, n, choice)
        assert int(acc.accept_len[r]) == want.accept_len
        nodes = acc.accept_nodes[r].cpu().numpy()
        toks = acc.accept_tokens[r].cpu().numpy()
        assert list(nodes[:want.accept_len]) == want.nodes and (nodes[want.accept_len:] == -1).all()
        assert list(toks[:want.accept_len]) == want.tokens and (toks[want.accept_len:] == -1).all()
        assert int(acc.bonus_token[r]) == want.bonus_token
        lens.append(want.accept_len)
    # the same call without node_choice: the library draws only at the rows the walk stands on (a cluster of
    # CTAs per request follows the walk); every output must be the same
    g2 = cases.Guard()
    lazy = dd.ddtree_accept_sampled(t, w.L, tok, par, n_rows, T, u, workspace=ws, out=cases.guarded_acceptance(g2, w.R, w.L, w.N),
                                    all_rows=False)
    g2.check()
    for name in ("accept_len", "accept_nodes", "accept_tokens", "bonus_token"):
        assert torch.equal(getattr(lazy, name), getattr(acc, name)), name
    return lens


def make_trees(w, variant="peak"):
    logits = cases.drafter_batch(w, variant)
    return cases.oracle_trees(w, logits, wl.root_tokens(w))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("T", [0.5, 1.0, 2.0])
def test_small_vocabulary(dtype, T):
    w = wl.small_workload(R=3, L=6, V=777, K=4, B=40, Hq=4, Hkv=2, d=64, dtype=dtype, prefix_lens=(5, 0, 9), index=70)
    trees = make_trees(w)
    tl = np.stack([wl.target_logits(w, trees[r].depth, r, "peak") for r in range(w.R)])
    ks = np.random.default_rng(int(T * 10)).integers(0, 2 ** 32, (w.R, w.N), dtype=np.uint64)
    ks[0, 0], ks[0, 1], ks[1, 0] = 0, 2 ** 32 - 1, 2 ** 31
    lens = run_and_compare(w, trees, tl, T, ks)
    if T == 0.5:
        assert max(lens) >= 1  # the boosted true tokens get accepted now and then


@pytest.mark.parametrize("dtype,V", [("f32", 20011), ("bf16", 70001)])
def test_several_chunks_and_a_ragged_tail(dtype, V):
    # the vocabulary spans several chunks of the passes; one row is all but deterministic, one has masked
    # (-inf) tokens, one has its mass at the very end of the vocabulary
    w = wl.small_workload(R=2, L=5, V=V, K=3, B=12, Hq=4, Hkv=2, d=64, dtype=dtype, prefix_lens=(3, 4), index=71)
    trees = make_trees(w)
    tl = np.stack([wl.target_logits(w, trees[r].depth, r, "peak") for r in range(w.R)])
    x = f32_rows(w, tl).copy()
    x[0, 1, :] = -50.0
    x[0, 1, V - 3] = 30.0
    x[0, 2, : V // 2] = -np.inf
    x[1, 0, :] = -20.0
    x[1, 0, V - 1] = 0.0
    x[1, 0, V - 2] = 0.0
    tl = wl.f32_to_bf16_bits(x) if dtype == "bf16" else x
    ks = np.random.default_rng(V).integers(0, 2 ** 32, (w.R, w.N), dtype=np.uint64)
    ks[1, 0] = 2 ** 32 - 1
    run_and_compare(w, trees, tl, 1.0, ks)


def test_low_temperature_is_the_greedy_walk():
    import paper_2604_12989_b200 as dd
    w = wl.small_workload(R=2, L=8, V=3000, K=4, B=64, Hq=4, Hkv=2, d=64, dtype="bf16", prefix_lens=(7, 8), index=72)
    trees = make_trees(w)
    tl = np.stack([wl.target_logits(w, trees[r].depth, r, "peak") for r in range(w.R)])
    ks = np.random.default_rng(1).integers(0, 2 ** 32, (w.R, w.N), dtype=np.uint64)
    lens = run_and_compare(w, trees, tl, 0.01, ks)
    t = aligned_rows(cases.to_torch(tl, True))
    tok = torch.from_numpy(np.stack([tr.token for tr in trees])).cuda()
    par = torch.from_numpy(np.stack([tr.parent for tr in trees])).cuda()
    n_rows = torch.tensor([tr.n_rows for tr in trees], dtype=torch.int32).cuda()
    greedy = dd.ddtree_accept(t, w.L, tok, par, n_rows)
    assert [int(v) for v in greedy.accept_len.cpu()] == lens


def test_full_vocabulary_on_the_benchmark_workload():
    # config 1 at full size (65 rows x 151936 bf16 logits), in the launch configuration a round would use
    w = wl.WORKLOADS[1]
    trees = make_trees(w, "lit")
    tl = np.stack([wl.target_logits(w, trees[r].depth, r, "lit") for r in range(w.R)])
    ks = np.random.default_rng(2).integers(0, 2 ** 32, (w.R, w.N), dtype=np.uint64)
    run_and_compare(w, trees, tl, 1.0, ks)


def test_argument_errors():
    import paper_2604_12989_b200 as dd
    w = wl.small_workload(R=1, L=4, V=300, K=2, B=8, Hq=2, Hkv=1, d=64, dtype="f32", prefix_lens=(3,), index=73)
    trees = make_trees(w)
    tl = np.stack([wl.target_logits(w, trees[0].depth, 0, "peak")])
    t = cases.to_torch(tl, False)
    tok = torch.from_numpy(trees[0].token[None]).cuda()
    par = torch.from_numpy(trees[0].parent[None]).cuda()
    n_rows = torch.tensor([trees[0].n_rows], dtype=torch.int32).cuda()
    u = torch.zeros(1, w.N, dtype=torch.int32).cuda()
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        with pytest.raises(dd.DDTreeError) as e:
            dd.ddtree_accept_sampled(t, w.L, tok, par, n_rows, bad, u)
        assert e.value.status == 1
    with pytest.raises(dd.DDTreeError):
        dd.ddtree_accept_sampled(t, w.L, tok, par, n_rows, 1.0, u, workspace=torch.empty(256, dtype=torch.uint8).cuda())


@pytest.mark.parametrize("seed", range(8))
def test_random_shapes(seed):
    rng = np.random.default_rng(100 + seed)
    R = int(rng.integers(1, 5))
    B = int(rng.choice([1, 2, 7, 16, 33, 64]))
    V = int(rng.choice([9, 64, 257, 4099, 8192, 8193, 16385]))
    K = int(min(V, rng.integers(1, 5)))
    dtype = str(rng.choice(["f32", "bf16"]))
    T = float(rng.choice([0.25, 0.9, 1.0, 3.0]))
    w = wl.small_workload(R=R, L=int(rng.integers(2, 9)), V=V, K=K, B=B, Hq=4, Hkv=2, d=64, dtype=dtype,
                          prefix_lens=tuple(int(x) for x in rng.integers(0, 20, R)), index=80 + seed)
    trees = make_trees(w)
    tl = np.stack([wl.target_logits(w, trees[r].depth, r, "peak") for r in range(w.R)])
    ks = rng.integers(0, 2 ** 32, (w.R, w.N), dtype=np.uint64)
    run_and_compare(w, trees, tl, T, ks)


# ---------------------------------------------------------------------------------------------
# The kernel against the rule itself (Section 4.4: the target's choice is a sample from its
# distribution at temperature T), not against the oracle's operation list: an inverse-CDF draw over
# the exact softmax, written out here in float64.
# ---------------------------------------------------------------------------------------------

def exact_inverse_cdf(x64, T, ks):
    """For every row: p = softmax(x / T) in float64, u = k / 2^32, the smallest v with cdf(v) > u, and the
    distance from u to the nearest cdf step on either side of that token (how close the draw was)."""
    z = x64 / T
    z = z - z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=1, keepdims=True)
    cdf = np.cumsum(p, axis=1)
    u = ks.astype(np.float64) / 2.0 ** 32
    choice = np.array([int(np.searchsorted(cdf[i], u[i], side="right")) for i in range(x64.shape[0])])
    choice = np.minimum(choice, x64.shape[1] - 1)
    hi = cdf[np.arange(len(u)), choice]
    lo = np.where(choice > 0, cdf[np.arange(len(u)), np.maximum(choice - 1, 0)], 0.0)
    return choice, np.minimum(np.abs(hi - u), np.abs(u - lo))


def drawn_tokens(w, trees, t_dev, T, ks):
    import paper_2604_12989_b200 as dd
    tok = torch.from_numpy(np.stack([tr.token for tr in trees])).cuda()
    par = torch.from_numpy(np.stack([tr.parent for tr in trees])).cuda()
    n_rows = torch.tensor([tr.n_rows for tr in trees], dtype=torch.int32).cuda()
    u = torch.from_numpy(ks.astype(np.uint32).view(np.int32)).cuda()
    acc = dd.ddtree_accept_sampled(t_dev, w.L, tok, par, n_rows, T, u)
    torch.cuda.synchronize()
    return acc.node_argmax.cpu().numpy()


@pytest.mark.parametrize("T", [0.7, 1.0, 1.5])
def test_draws_equal_the_exact_inverse_cdf_at_full_vocabulary(T):
    """Config 1's target logits (65 rows x 151936 bf16 values), as many sets of random inputs per temperature
    as it takes to compare more than 1000 draws.  Every draw whose u is further than 1e-5 from a step of the exact
    cdf must give the exact token (the fixed-point weights are within 5e-6 of the exact numerators, so the
    two cdfs differ by less than that everywhere)."""
    w = wl.WORKLOADS[1]
    trees = make_trees(w, "peak")
    tl = np.stack([wl.target_logits(w, trees[r].depth, r, "peak") for r in range(w.R)])
    x64 = wl.bf16_to_f64(tl[0])
    t_dev = aligned_rows(cases.to_torch(tl, True))
    n = trees[0].n_rows
    compared = 0
    for rep in range(96):
        if compared >= 1000:
            break
        ks = np.random.default_rng([int(T * 100), rep]).integers(0, 2 ** 32, (w.R, w.N), dtype=np.uint64)
        got = drawn_tokens(w, trees, t_dev, T, ks)[0, :n]
        want, margin = exact_inverse_cdf(x64[:n], T, ks[0, :n])
        clear = margin >= 1e-5
        np.testing.assert_array_equal(got[clear], want[clear])
        compared += int(clear.sum())
    assert compared >= 1000


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_draw_frequencies_follow_the_softmax(dtype):
    """Many rows with the same logits and independent random inputs: the empirical token frequencies of the
    GPU draws match softmax(x / T) within five standard errors, and the draws are the exact inverse-CDF
    tokens wherever u is clear of a cdf step."""
    V, T = 48, 1.3
    w = wl.small_workload(R=8, L=8, V=V, K=4, B=1024, Hq=4, Hkv=2, d=64, dtype=dtype, prefix_lens=tuple([2] * 8), index=74)
    trees = make_trees(w)
    rng = np.random.default_rng(74)
    row = (rng.standard_normal(V) * 2.0).astype(np.float32)
    row = wl.round_through_bf16(row)  # exactly representable in both dtypes
    x = np.broadcast_to(row, (w.R, w.N, V)).copy()
    tl = wl.f32_to_bf16_bits(x) if dtype == "bf16" else x
    ks = rng.integers(0, 2 ** 32, (w.R, w.N), dtype=np.uint64)
    got = drawn_tokens(w, trees, aligned_rows(cases.to_torch(tl, dtype == "bf16")), T, ks)
    draws, wants, margins = [], [], []
    for r in range(w.R):
        n = trees[r].n_rows
        draws.append(got[r, :n])
        want, margin = exact_inverse_cdf(x[r, :n].astype(np.float64), T, ks[r, :n])
        wants.append(want)
        margins.append(margin)
    draws, wants, margins = np.concatenate(draws), np.concatenate(wants), np.concatenate(margins)
    assert len(draws) >= 2000
    clear = margins >= 1e-5
    np.testing.assert_array_equal(draws[clear], wants[clear])
    z = row.astype(np.float64) / T
    p = np.exp(z - z.max())
    p /= p.sum()
    freq = np.bincount(draws, minlength=V) / len(draws)
    se = np.sqrt(p * (1 - p) / len(draws))
    assert (np.abs(freq - p) <= 5 * se + 1e-4).all(), np.abs(freq - p).max()
