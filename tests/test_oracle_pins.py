"""Pins for the CPU oracle: every function is checked against something other
than itself -- the paper's Figure 2, closed forms, brute-force enumeration, or a
library routine -- chosen so that a dropped term, a wrong sign or index, or a
transposed operand fails at least one test.  CPU only."""
import itertools
import math

import numpy as np
import pytest
import scipy.special
import torch

from oracle import ddtree_oracle as orc


# ----------------------------------------------------------------------------
# helpers (independent re-derivations, no oracle code)
# ----------------------------------------------------------------------------

def random_logits(rng, L, V, scale=2.0):
    return rng.standard_normal((L, V)) * scale


def brute_force_prefixes(q, ranks_allowed=None):
    """All non-empty prefixes u (tuples of token ids) of length <= L with their
    probability prod_i q[i][u_i] (Eq. for q(u | c, b) in Section 4.2)."""
    L, V = q.shape
    out = []
    for d in range(1, L + 1):
        for u in itertools.product(range(V), repeat=d):
            if ranks_allowed is not None and any(u[i] not in ranks_allowed[i] for i in range(d)):
                continue
            out.append((math.prod(q[i, u[i]] for i in range(d)), u))
    return out


def tree_token_paths(ct):
    """Set of token-id tuples (root path without the root) of a compiled tree."""
    paths = set()
    for i in range(1, ct.n_rows):
        u, j = [], i
        while j != 0:
            u.append(int(ct.token[j]))
            j = int(ct.parent[j])
        paths.add(tuple(reversed(u)))
    return paths


def parse_ints(s):
    return [int(t) for t in s.split()]


# ----------------------------------------------------------------------------
# log-softmax and top-K
# ----------------------------------------------------------------------------

def test_log_softmax_matches_scipy_and_normalises():
    rng = np.random.default_rng(1)
    x = random_logits(rng, 5, 97, 4.0)
    got = orc.log_softmax(x)
    np.testing.assert_allclose(got, scipy.special.log_softmax(x, axis=-1), rtol=0, atol=1e-13)
    np.testing.assert_allclose(np.exp(got).sum(-1), 1.0, atol=1e-13)
    # adding a per-row constant changes nothing
    np.testing.assert_allclose(orc.log_softmax(x + rng.standard_normal((5, 1)) * 50), got, atol=1e-12)
    # large logits must not overflow
    big = np.array([[1000.0, 999.0, 0.0]])
    assert np.isfinite(orc.log_softmax(big)).all()
    np.testing.assert_allclose(orc.log_softmax(big)[0, 0], -math.log(1 + math.exp(-1) + math.exp(-1000)), atol=1e-12)


def test_log_softmax_uniform_closed_form():
    np.testing.assert_allclose(orc.log_softmax(np.full((2, 8), 3.25)), -math.log(8), atol=1e-15)


def test_top_k_against_python_sort_with_ties():
    rng = np.random.default_rng(2)
    # values on a coarse lattice so ties are common
    x = np.round(rng.standard_normal((6, 40)) * 2) / 2
    tok, lq = orc.top_k(x, 7)
    for i in range(6):
        want = sorted(range(40), key=lambda v: (-x[i, v], v))[:7]
        assert list(tok[i]) == want
        np.testing.assert_allclose(lq[i], scipy.special.log_softmax(x[i])[want], atol=1e-13)
        assert (np.diff(lq[i]) <= 0).all()


def test_top_k_rejects_bad_k():
    with pytest.raises(ValueError):
        orc.top_k(np.zeros((2, 3)), 4)


# ----------------------------------------------------------------------------
# Figure 2 worked example
# ----------------------------------------------------------------------------

def fig2_logits(fx):
    V, L = int(fx["V"]), int(fx["L"])
    x = np.zeros((L, V))
    for i in range(L):
        q = [float(t) for t in fx[f"q_by_rank_{i + 1}"].split()]
        tok = parse_ints(fx[f"tok_by_rank_{i + 1}"])
        assert abs(sum(q) - 1) < 1e-12
        for r in range(V):
            x[i, tok[r]] = math.log(q[r]) + 0.37 * (i + 1)  # per-row constants must not matter
    return x


def test_fig2_fixture_is_the_top8_by_brute_force(fig2):
    """The fixture's distributions really induce Figure 2(a): enumerate all 84 prefixes."""
    x = fig2_logits(fig2)
    q = np.exp(scipy.special.log_softmax(x, axis=-1))
    allp = sorted(brute_force_prefixes(q), key=lambda t: -t[0])
    assert len(allp) == 84
    B = int(fig2["B"])
    assert allp[B - 1][0] - allp[B][0] > 1e-3  # unique top-8
    top = {u for _, u in allp[:B]}
    tok = [parse_ints(fig2[f"tok_by_rank_{i + 1}"]) for i in range(3)]
    want = set()
    for r in fig2["rho"].split()[1:]:
        ranks = [int(t) for t in r.strip("()").split(",") if t]
        want.add(tuple(tok[i][ranks[i] - 1] for i in range(len(ranks))))
    assert top == want


def test_fig2_tree_arrays(fig2):
    x = fig2_logits(fig2)
    ct = orc.build(x, int(fig2["K"]), int(fig2["B"]), int(fig2["root_token"]), int(fig2["prefix_len"]))
    assert ct.n_rows == 9
    assert list(ct.parent) == parse_ints(fig2["parent"])
    assert list(ct.depth) == parse_ints(fig2["depth"])
    assert list(ct.token) == parse_ints(fig2["token"])
    assert list(ct.position_ids) == [int(fig2["prefix_len"]) + d for d in parse_ints(fig2["depth"])]
    assert [int(m[0]) for m in ct.mask] == [int(h, 16) for h in fig2["mask_hex"].split()]
    assert list(ct.first_child) == parse_ints(fig2["first_child"])
    assert list(ct.child_count) == parse_ints(fig2["child_count"])
    got_rho = ["(" + ",".join(str(t) for t in r) + ")" for r in ct.rho]
    assert got_rho == fig2["rho"].split()


def test_fig2_walk(fig2):
    x = fig2_logits(fig2)
    ct = orc.build(x, int(fig2["K"]), int(fig2["B"]), int(fig2["root_token"]), int(fig2["prefix_len"]))
    acc = orc.accept_walk(ct.token, ct.parent, ct.n_rows, np.array(parse_ints(fig2["choice"])))
    assert acc.accept_len == int(fig2["accept_len"])
    assert acc.nodes == parse_ints(fig2["accept_nodes"])
    assert acc.tokens == parse_ints(fig2["accept_tokens"])
    assert acc.bonus_token == int(fig2["bonus_token"])


def test_rank_tuple_convention():
    """Section 4.3's example: rho = (1,3,2) is the best token at position 1, the third best
    at position 2, the second best at position 3."""
    x = np.array([[0.0, 5.0, 1.0, 2.0], [9.0, 1.0, 4.0, 6.0], [3.0, 2.0, 8.0, 7.0]])
    tok, lq = orc.top_k(x, 4)
    nodes, _ = orc.best_first_tree(lq, 4 + 16 + 64)  # exhaust S_K
    ct = orc.compile_tree(nodes, tok, 0, 0, 84)
    row = ct.rho.index((1, 3, 2))
    path = []
    j = row
    while j:
        path.append(int(ct.token[j]))
        j = int(ct.parent[j])
    assert path[::-1] == [1, 2, 3]
    want = scipy.special.log_softmax(x, axis=-1)
    np.testing.assert_allclose(ct.logprob[row], want[0, 1] + want[1, 2] + want[2, 3], atol=1e-12)


# ----------------------------------------------------------------------------
# Algorithm 1 vs the definition (Propositions 1-3, Lemma 1)
# ----------------------------------------------------------------------------

@pytest.mark.parametrize("V,L,B,seed", [(3, 3, 5, 0), (4, 3, 9, 1), (5, 4, 17, 2), (6, 3, 30, 3), (4, 4, 50, 4),
                                        (2, 4, 7, 5), (5, 2, 6, 6)])
def test_heap_equals_brute_force_top_b(V, L, B, seed):
    rng = np.random.default_rng(seed)
    x = random_logits(rng, L, V)
    q = np.exp(scipy.special.log_softmax(x, axis=-1))
    K = min(B, V)  # the paper's K
    ct = orc.build(x, K, B, 0, 0)
    allp = sorted(brute_force_prefixes(q), key=lambda t: -t[0])
    nB = min(B, len(allp))
    assert ct.n_rows - 1 == nB
    if nB < len(allp):
        assert allp[nB - 1][0] > allp[nB][0]  # unique cut for this seed
    assert tree_token_paths(ct) == {u for _, u in allp[:nB]}
    # node log-probabilities are the log of the brute-force products
    prob = {u: p for p, u in allp}
    for i in range(1, ct.n_rows):
        u, j = [], i
        while j:
            u.append(int(ct.token[j]))
            j = int(ct.parent[j])
        np.testing.assert_allclose(ct.logprob[i], math.log(prob[tuple(reversed(u))]), atol=1e-12)


@pytest.mark.parametrize("V,L,B,K,seed", [(5, 3, 10, 2, 0), (6, 4, 20, 3, 1), (6, 3, 14, 2, 2)])
def test_heap_with_small_k_is_top_b_of_S_K(V, L, B, K, seed):
    """With K < min(B, V) Algorithm 1 returns the top-B of S_K (proof of Proposition 3)."""
    rng = np.random.default_rng(seed)
    x = random_logits(rng, L, V)
    q = np.exp(scipy.special.log_softmax(x, axis=-1))
    allowed = [set(sorted(range(V), key=lambda v: (-x[i, v], v))[:K]) for i in range(L)]
    allp = sorted(brute_force_prefixes(q, allowed), key=lambda t: -t[0])
    ct = orc.build(x, K, B, 0, 0)
    nB = min(B, len(allp))
    assert ct.n_rows - 1 == nB
    assert tree_token_paths(ct) == {u for _, u in allp[:nB]}


@pytest.mark.parametrize("seed", range(6))
def test_pop_order_properties(seed):
    """Proof of Proposition 3: pops are non-increasing in sigma; every tuple pops after its
    predecessor (previous sibling, or parent for rank 1); the result is prefix-closed."""
    rng = np.random.default_rng(seed)
    x = random_logits(rng, 6, 50, 3.0)
    tok, lq = orc.top_k(x, 8)
    nodes, left = orc.best_first_tree(lq, 40)
    sig = [n.sigma for n in nodes]
    assert all(a >= b for a, b in zip(sig, sig[1:]))
    assert left is not None and left <= sig[-1]
    seen = set()
    for n in nodes:
        r = n.rho
        if r != (1,):
            pred = r[:-1] + (r[-1] - 1,) if r[-1] > 1 else r[:-1]
            assert pred in seen
        if len(r) > 1:
            assert r[:-1] in seen  # prefix-closed
        np.testing.assert_allclose(n.sigma, sum(lq[i, r[i] - 1] for i in range(len(r))), atol=1e-12)
        seen.add(r)
    assert len(seen) == 40


@pytest.mark.parametrize("seed", range(4))
def test_prop1_sum_of_prefix_mass_is_expected_acceptance(seed):
    """Proposition 1: E_{Y~Q}[alpha_T(Y)] = sum_{u in T} q(u), by enumerating all V^L sequences."""
    rng = np.random.default_rng(seed)
    V, L, B = 4, 4, 11
    x = random_logits(rng, L, V)
    q = np.exp(scipy.special.log_softmax(x, axis=-1))
    ct = orc.build(x, min(B, V), B, 0, 0)
    paths = tree_token_paths(ct)
    expect = 0.0
    for y in itertools.product(range(V), repeat=L):
        alpha = 0
        for d in range(1, L + 1):
            if tuple(y[:d]) in paths:
                alpha = d
            else:
                break
        expect += alpha * math.prod(q[i, y[i]] for i in range(L))
    np.testing.assert_allclose(np.exp(ct.logprob[1:ct.n_rows]).sum(), expect, atol=1e-12)


def test_fig2_objective_value(fig2):
    x = fig2_logits(fig2)
    ct = orc.build(x, 4, 8, 0, 0)
    np.testing.assert_allclose(np.exp(ct.logprob[1:9]).sum(), 1.94168, atol=1e-9)


@pytest.mark.parametrize("seed", range(4))
def test_lemma1_k_equal_b_same_as_k_equal_v(seed):
    rng = np.random.default_rng(seed)
    x = random_logits(rng, 5, 64, 3.0)
    B = 12
    a = orc.build(x, B, B, 3, 0)
    b = orc.build(x, 64, B, 3, 0)
    assert list(a.token) == list(b.token) and list(a.parent) == list(b.parent)


@pytest.mark.parametrize("seed", range(4))
def test_trees_nest_as_budget_grows(seed):
    rng = np.random.default_rng(seed)
    x = random_logits(rng, 6, 30, 3.0)
    prev = set()
    for B in range(1, 25):
        cur = tree_token_paths(orc.build(x, 8, B, 0, 0))
        assert prev <= cur and len(cur) == B
        prev = cur


def test_dflash_special_case_single_trajectory():
    """K = 1 and B = L: the tree is the single chain of per-position argmaxes (vanilla DFlash)."""
    rng = np.random.default_rng(7)
    L, V = 8, 200
    x = random_logits(rng, L, V, 3.0)
    ct = orc.build(x, 1, L, 11, 100)
    assert ct.n_rows == L + 1
    assert list(ct.token[1:]) == list(np.argmax(x, axis=-1))
    assert list(ct.parent) == [-1] + list(range(L))
    assert list(ct.depth) == list(range(L + 1))
    assert list(ct.position_ids) == [100 + d for d in range(L + 1)]


def test_heap_runs_empty_when_budget_exceeds_S_K():
    """Algorithm 1 stops when the heap is empty: K = 1, B > L gives L nodes; in general |S_K|."""
    rng = np.random.default_rng(8)
    x = random_logits(rng, 4, 10)
    ct = orc.build(x, 1, 9, 0, 0)
    assert ct.n_rows == 5
    assert (ct.token[5:] == -1).all() and (ct.parent[5:] == -1).all() and (ct.mask[5:] == 0).all()
    ct = orc.build(x[:3], 2, 100, 0, 0)
    assert ct.n_rows == 1 + 2 + 4 + 8


def test_budget_counts_nodes_not_root():
    rng = np.random.default_rng(9)
    ct = orc.build(random_logits(rng, 4, 10), 4, 6, 42, 5)
    assert ct.n_rows == 7 and ct.token[0] == 42 and ct.parent[0] == -1 and ct.position_ids[0] == 5


@pytest.mark.parametrize("seed", range(4))
def test_compile_invariants(seed):
    rng = np.random.default_rng(seed)
    B = 70  # spans three mask words
    x = random_logits(rng, 8, 300, 3.0)
    ct = orc.build(x, 8, B, 1, 1000)
    n = ct.n_rows
    assert n == B + 1
    for i in range(1, n):
        p = ct.parent[i]
        assert 0 <= p < i
        assert ct.depth[i] == ct.depth[p] + 1
        bits = [j for j in range(n) if (int(ct.mask[i, j // 32]) >> (j % 32)) & 1]
        chain, j = [], i
        while j >= 0:
            chain.append(j)
            j = ct.parent[j]
        assert bits == sorted(chain)
        assert len(bits) == ct.depth[i] + 1
    # level order, siblings adjacent with distinct tokens
    keys = [(len(r), r) for r in ct.rho[:n]]
    assert keys == sorted(keys)
    for p in range(n):
        kids = [j for j in range(n) if ct.parent[j] == p]
        assert ct.child_count[p] == len(kids)
        if kids:
            assert ct.first_child[p] == kids[0] and kids == list(range(kids[0], kids[0] + len(kids)))
            assert len({int(ct.token[j]) for j in kids}) == len(kids)
        else:
            assert ct.first_child[p] == -1


# ----------------------------------------------------------------------------
# tree attention
# ----------------------------------------------------------------------------

def attention_case(seed, P, B=20, Hq=4, Hkv=2, d=16, L=6, V=50, K=4):
    rng = np.random.default_rng(seed)
    ct = orc.build(random_logits(rng, L, V, 3.0), K, B, 0, P)
    N = B + 1
    q = rng.standard_normal((N, Hq, d))
    kp, vp = rng.standard_normal((P, Hkv, d)), rng.standard_normal((P, Hkv, d))
    kt, vt = rng.standard_normal((N, Hkv, d)), rng.standard_normal((N, Hkv, d))
    return ct, q, kp, vp, kt, vt


@pytest.mark.parametrize("P", [0, 1, 7, 33])
def test_tree_attention_equals_plain_attention_over_root_path(P):
    """Section 4.4: a node sees the cached context, the root, its ancestors and itself, i.e. the
    sequence it would see if only its own root path had been drafted.  The path is re-derived
    from parent[] (not from the mask) and fed to torch's unmasked attention as a library pin."""
    ct, q, kp, vp, kt, vt = attention_case(3 + P, P)
    Hq, Hkv = q.shape[1], kt.shape[1]
    G = Hq // Hkv
    out, lse = orc.tree_attention(q, kp, vp, kt, vt, ct.mask, ct.n_rows)
    for i in range(ct.n_rows):
        chain, j = [], i
        while j >= 0:
            chain.append(j)
            j = int(ct.parent[j])
        chain = chain[::-1]
        for h in range(Hq):
            kv = h // G
            ks = torch.from_numpy(np.concatenate([kp[:, kv], kt[chain, kv]]))[None, None]
            vs = torch.from_numpy(np.concatenate([vp[:, kv], vt[chain, kv]]))[None, None]
            qs = torch.from_numpy(q[i, h])[None, None, None]
            ref = torch.nn.functional.scaled_dot_product_attention(qs, ks, vs)[0, 0, 0].numpy()
            np.testing.assert_allclose(out[i, h], ref, atol=1e-12)
            s = (ks[0, 0].numpy() @ q[i, h]) / math.sqrt(q.shape[2])
            np.testing.assert_allclose(lse[i, h], scipy.special.logsumexp(s), atol=1e-12)


def test_chain_tree_is_causal_attention():
    """A chain (K = 1) under the ancestor mask is ordinary causal attention of N new tokens."""
    rng = np.random.default_rng(5)
    L, Hq, Hkv, d, P = 7, 4, 2, 8, 5
    ct = orc.build(random_logits(rng, L, 30), 1, L, 0, P)
    N = L + 1
    q = rng.standard_normal((N, Hq, d))
    kp, vp = rng.standard_normal((P, Hkv, d)), rng.standard_normal((P, Hkv, d))
    kt, vt = rng.standard_normal((N, Hkv, d)), rng.standard_normal((N, Hkv, d))
    out, _ = orc.tree_attention(q, kp, vp, kt, vt, ct.mask, ct.n_rows)
    keys = torch.from_numpy(np.concatenate([kp, kt]).transpose(1, 0, 2)).repeat_interleave(Hq // Hkv, 0)[None]
    vals = torch.from_numpy(np.concatenate([vp, vt]).transpose(1, 0, 2)).repeat_interleave(Hq // Hkv, 0)[None]
    qq = torch.from_numpy(q.transpose(1, 0, 2))[None]
    causal = torch.ones(N, P + N, dtype=torch.bool).tril(diagonal=P)
    ref = torch.nn.functional.scaled_dot_product_attention(qq, keys, vals, attn_mask=causal)[0]
    np.testing.assert_allclose(out, ref.numpy().transpose(1, 0, 2), atol=1e-12)


def test_zero_query_gives_mean_of_visible_values():
    ct, q, kp, vp, kt, vt = attention_case(11, 9)
    q[:] = 0
    out, lse = orc.tree_attention(q, kp, vp, kt, vt, ct.mask, ct.n_rows)
    for i in range(ct.n_rows):
        chain, j = [], i
        while j >= 0:
            chain.append(j)
            j = int(ct.parent[j])
        for h in range(q.shape[1]):
            kv = h // 2
            mean = (vp[:, kv].sum(0) + vt[chain, kv].sum(0)) / (9 + ct.depth[i] + 1)
            np.testing.assert_allclose(out[i, h], mean, atol=1e-12)
            np.testing.assert_allclose(lse[i, h], math.log(9 + ct.depth[i] + 1), atol=1e-12)


def test_scale_and_subset_arguments():
    ct, q, kp, vp, kt, vt = attention_case(12, 4)
    full, _ = orc.tree_attention(q, kp, vp, kt, vt, ct.mask, ct.n_rows)
    sub, _ = orc.tree_attention(q, kp, vp, kt, vt, ct.mask, ct.n_rows, rows=[3, 7], heads=[1, 2])
    np.testing.assert_array_equal(sub, full[[3, 7]][:, [1, 2]])
    d = q.shape[2]
    scaled, _ = orc.tree_attention(q * 2, kp, vp, kt, vt, ct.mask, ct.n_rows, scale=0.5 / math.sqrt(d))
    np.testing.assert_allclose(scaled, full, atol=1e-12)


# ----------------------------------------------------------------------------
# argmax and walk
# ----------------------------------------------------------------------------

def test_node_argmax_lowest_id_on_ties():
    x = np.array([[1.0, 3.0, 3.0, 2.0], [5.0, 5.0, 5.0, 5.0], [-1.0, -2.0, -0.5, -0.5]])
    assert list(orc.node_argmax(x)) == [1, 0, 2]


def brute_force_longest_match(token, parent, n_rows, choice):
    best = (0, 0)
    for i in range(n_rows):
        chain, j = [], i
        while j >= 0:
            chain.append(j)
            j = int(parent[j])
        chain = chain[::-1]
        if all(token[chain[k]] == choice[chain[k - 1]] for k in range(1, len(chain))):
            best = max(best, (len(chain) - 1, i))
    return best


@pytest.mark.parametrize("seed", range(12))
def test_walk_equals_brute_force_longest_match(seed):
    rng = np.random.default_rng(seed)
    L, V, K, B = 6, 12, 4, 40
    ct = orc.build(random_logits(rng, L, V, 1.0), K, B, 0, 0)
    # target choices that often hit drafted children (small vocabulary), sometimes via rank >= 2
    choice = rng.integers(0, V, B + 1).astype(np.int32)
    for i in range(ct.n_rows):
        if ct.child_count[i] and rng.random() < 0.7:
            choice[i] = ct.token[ct.first_child[i] + rng.integers(0, ct.child_count[i])]
    acc = orc.accept_walk(ct.token, ct.parent, ct.n_rows, choice)
    want_len, want_node = brute_force_longest_match(ct.token, ct.parent, ct.n_rows, choice)
    assert acc.accept_len == want_len
    assert (acc.nodes[-1] if acc.nodes else 0) == want_node
    assert acc.bonus_token == choice[want_node]
    assert acc.tokens == [int(ct.token[j]) for j in acc.nodes]
    assert all(ct.parent[b] == a for a, b in zip([0] + acc.nodes, acc.nodes))


def test_walk_stops_at_leaf_of_full_depth():
    rng = np.random.default_rng(3)
    L = 4
    ct = orc.build(random_logits(rng, L, 9), 1, L, 0, 0)
    choice = np.concatenate([ct.token[1:], [5]]).astype(np.int32)
    acc = orc.accept_walk(ct.token, ct.parent, ct.n_rows, choice)
    assert acc.accept_len == L and acc.nodes == [1, 2, 3, 4] and acc.bonus_token == 5


@pytest.mark.parametrize("seed", range(6))
def test_compacted_cache_is_the_context_the_last_accepted_node_saw(seed):
    """Section 4.4: after the walk only the accepted path stays cached.  Pinned on the attention
    itself: the last accepted node attended to prefix + root + ancestors + itself, so plain
    unmasked attention (torch SDPA) of its query over the first P + accept_len + 1 rows of the
    compacted cache must give its tree-attention output, and every moved row must sit at the
    position id it was verified at."""
    rng = np.random.default_rng(100 + seed)
    L, V, K, B, P, Hq, Hkv, d = 6, 12, 3, 30, 5 + seed, 4, 2, 8
    ct = orc.build(random_logits(rng, L, V, 1.0), K, B, 0, P)
    choice = rng.integers(0, V, B + 1).astype(np.int32)
    for i in range(ct.n_rows):  # make long accepted paths likely
        if ct.child_count[i] and rng.random() < 0.85:
            choice[i] = ct.token[ct.first_child[i] + rng.integers(0, ct.child_count[i])]
    acc = orc.accept_walk(ct.token, ct.parent, ct.n_rows, choice)
    N = B + 1
    q = rng.standard_normal((N, Hq, d))
    cap = P + L + 1
    kc, vc = rng.standard_normal((cap, Hkv, d)), rng.standard_normal((cap, Hkv, d))
    kt, vt = rng.standard_normal((N, Hkv, d)), rng.standard_normal((N, Hkv, d))
    out, _ = orc.tree_attention(q, kc[:P], vc[:P], kt, vt, ct.mask, ct.n_rows)
    k2 = orc.kv_compact(kc, kt, P, acc.nodes)
    v2 = orc.kv_compact(vc, vt, P, acc.nodes)
    np.testing.assert_array_equal(k2[:P], kc[:P])                       # the context is untouched
    np.testing.assert_array_equal(k2[P + acc.accept_len + 1:], kc[P + acc.accept_len + 1:])
    last = acc.nodes[-1] if acc.nodes else 0
    n_ctx = P + acc.accept_len + 1
    for h in range(Hq):
        kv = h // (Hq // Hkv)
        ks = torch.from_numpy(k2[:n_ctx, kv])[None, None]
        vs = torch.from_numpy(v2[:n_ctx, kv])[None, None]
        ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q[last, h])[None, None, None], ks, vs)
        np.testing.assert_allclose(out[last, h], ref[0, 0, 0].numpy(), atol=1e-12)
    for i, j in enumerate([0] + acc.nodes):
        assert ct.position_ids[j] == P + i  # cache row P + i holds the token verified at position P + i


# --------------------------------------------------------------------------
# Section 4.4 with the temperature-based decoding rule: fixed-point inverse-CDF draw
# --------------------------------------------------------------------------

def _exact_softmax(x, T):
    z = (np.asarray(x, np.float64) - float(np.max(x))) / T
    e = np.exp(z)
    return e, e / e.sum()


@pytest.mark.parametrize("T", [0.3, 1.0, 2.5])
def test_sampling_weights_are_the_softmax_numerators(T):
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(3000) * 4).astype(np.float32)
    x[7] = -np.inf                                          # a masked token never gets weight
    w = np.array(orc.sampling_weights(x, T), dtype=np.float64) / 2.0 ** 40
    e, _ = _exact_softmax(x, T)
    assert w[7] == 0 and w[int(np.argmax(x))] == 1.0        # the maximum has weight exactly 2^40
    assert np.all(np.abs(w - e) <= 2.0 ** -40 + 5e-6 * e)
    assert np.all(w[e < 2.0 ** -41] <= 2.0 ** -40)          # negligible tokens get (almost) nothing


def test_sample_token_equals_the_exact_inverse_cdf_away_from_boundaries():
    rng = np.random.default_rng(6)
    agree = tested = 0
    for trial in range(60):
        V = int(rng.integers(2, 400))
        x = (rng.standard_normal(V) * 3).astype(np.float32)
        T = float(rng.choice([0.5, 1.0, 1.7]))
        _, p = _exact_softmax(x, T)
        cdf = np.cumsum(p)
        for k in rng.integers(0, 2 ** 32, 25):
            u = int(k) / 2.0 ** 32
            if np.min(np.abs(cdf - u)) < 1e-5:              # the two may differ when u sits on a boundary
                continue
            tested += 1
            agree += orc.sample_token(x, T, int(k)) == int(np.searchsorted(cdf, u, side="right"))
    assert tested > 1000 and agree == tested


def test_sample_token_on_tiny_rows_by_exact_rational_arithmetic():
    # weights that are exact powers of two: logits k*ln2*T apart give e_v = 2^-k, no rounding anywhere
    from fractions import Fraction
    x = np.array([0.0, -1.0, -3.0, 0.0, -2.0], np.float32)  # with c = 1: weights 1, 1/2, 1/8, 1, 1/4
    T = 1.4426950408889634                                   # log2(e) / T == 1.0f exactly
    w = orc.sampling_weights(x, T)
    assert w == [2 ** 40, 2 ** 39, 2 ** 37, 2 ** 40, 2 ** 38]
    total = Fraction(sum(w))
    for k in [0, 1, 2 ** 31, 2 ** 32 - 1] + [int(v) for v in np.random.default_rng(7).integers(0, 2 ** 32, 200)]:
        u = Fraction(k, 2 ** 32)
        acc = Fraction(0)
        for v, wv in enumerate(w):
            acc += Fraction(wv) / total
            if acc > u:
                break
        assert orc.sample_token(x, T, k) == v


def test_sample_token_limits_and_monotonicity():
    rng = np.random.default_rng(8)
    x = (rng.standard_normal(500) * 2).astype(np.float32)
    x[:3] = -np.inf
    x[-2:] = -200.0                                          # weight 0 at T = 1
    assert orc.sample_token(x, 1.0, 0) == 3                  # first token with weight
    assert orc.sample_token(x, 1.0, 2 ** 32 - 1) == 497      # last token with weight
    ks = np.sort(rng.integers(0, 2 ** 32, 300))
    toks = [orc.sample_token(x, 1.0, int(k)) for k in ks]
    assert toks == sorted(toks)                              # the draw is monotone in u
    # T -> 0: the draw is the arg-max whatever u is
    for k in rng.integers(0, 2 ** 32, 20):
        assert orc.sample_token(x, 1e-3, int(k)) == int(np.argmax(x))


def test_sample_token_frequencies_follow_softmax():
    rng = np.random.default_rng(9)
    x = np.array([1.0, 0.0, -1.0, 2.0, 0.5, -3.0, 1.5, 0.0], np.float32)
    T = 0.8
    _, p = _exact_softmax(x, T)
    n = 20000
    counts = np.bincount([orc.sample_token(x, T, int(k)) for k in rng.integers(0, 2 ** 32, n)], minlength=8)
    sigma = np.sqrt(n * p * (1 - p))
    assert np.all(np.abs(counts - n * p) <= 4.5 * sigma + 1)


def test_sampled_walk_reduces_to_the_greedy_walk_at_low_temperature():
    rng = np.random.default_rng(10)
    logits = rng.standard_normal((6, 50))
    tree = orc.build(logits, 4, 20, root_token=3, prefix_len=11)
    target = (rng.standard_normal((tree.n_rows, 50)) * 2).astype(np.float32)
    for i in range(tree.n_rows):                             # make the target agree with some child now and then
        kids = [j for j in range(tree.n_rows) if tree.parent[j] == i]
        if kids and i % 2 == 0:
            target[i, tree.token[kids[0]]] = 9.0
    greedy = orc.accept_walk(tree.token, tree.parent, tree.n_rows, orc.node_argmax(target))
    ks = rng.integers(0, 2 ** 32, tree.n_rows)
    cold = orc.accept_walk(tree.token, tree.parent, tree.n_rows, orc.node_sampled(target, 1e-3, ks))
    assert (cold.accept_len, cold.nodes, cold.bonus_token) == (greedy.accept_len, greedy.nodes, greedy.bonus_token)
    assert greedy.accept_len >= 1


# --------------------------------------------------------------------------
# Rotary positional encoding at the tree's position ids
# --------------------------------------------------------------------------

def test_rope_against_the_real_valued_textbook_form():
    rng = np.random.default_rng(20)
    x = rng.standard_normal((5, 3, 8))
    pos = np.array([0, 1, 7, 100, 4097])
    out = orc.rope(x, pos, 10000.0)
    for r in range(5):
        for j in range(4):
            a = pos[r] * 10000.0 ** (-2.0 * j / 8)
            c, s = math.cos(a), math.sin(a)
            np.testing.assert_allclose(out[r, :, j], x[r, :, j] * c - x[r, :, j + 4] * s, atol=1e-12)
            np.testing.assert_allclose(out[r, :, j + 4], x[r, :, j + 4] * c + x[r, :, j] * s, atol=1e-12)
    np.testing.assert_array_equal(out[0], x[0])                     # position 0 is the identity


def test_rope_preserves_norms_and_makes_scores_depend_on_the_distance_only():
    rng = np.random.default_rng(21)
    q, k = rng.standard_normal((1, 1, 64)), rng.standard_normal((1, 1, 64))
    np.testing.assert_allclose(np.linalg.norm(orc.rope(q, [12345], 1e6)), np.linalg.norm(q), rtol=1e-12)
    dots = [float(np.sum(orc.rope(q, [m], 1e6) * orc.rope(k, [m - 9], 1e6))) for m in (9, 50, 4000)]
    np.testing.assert_allclose(dots, dots[0], rtol=1e-9)            # <R_m q, R_n k> is a function of m - n
    # composition: rotating by m and then by n is rotating by m + n
    np.testing.assert_allclose(orc.rope(orc.rope(q, [30], 1e6), [12], 1e6), orc.rope(q, [42], 1e6), atol=1e-12)
