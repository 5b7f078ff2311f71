"""Several decoding rounds in a closed loop on the GPU against the same loop over the CPU oracle
(Section 4.1: every round starts from the bonus token of the round before; Section 4.4: after the walk the
accepted path's keys and values join the cache).  Round t+1 uses what round t produced: its root is round
t's bonus token, its prefix has grown by accept_len + 1, and its attention reads the cache rows round t's
compaction wrote.  Every round: tree arrays, acceptance and bonus token bit for bit, attention of every layer
within tolerance, the caches bit for bit after compaction."""
import numpy as np
import pytest
import torch

from oracle import ddtree_oracle as orc
from paper_2604_12989_b200 import workloads as wl
from tests import ddtree_cases as cases

pytestmark = pytest.mark.gpu


def bf16_normal(rng, *shape):
    return wl.f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))


@pytest.mark.parametrize("temperature", [0.0, 0.8])
def test_four_rounds_of_two_requests_match_the_oracle_loop(temperature):
    import paper_2604_12989_b200 as dd
    R, L, V, K, B, Hq, Hkv, d, layers, rounds = 2, 6, 2000, 4, 40, 8, 2, 128, 2, 4
    start = (150, 37)
    cap = [p + rounds * (L + 1) for p in start]          # cache rows a request may ever hold
    rng = np.random.default_rng(11)
    # one cache slab per layer and request, the first P rows filled
    slabs_k = [[bf16_normal(rng, cap[r], Hkv, d) for r in range(R)] for _ in range(layers)]
    slabs_v = [[bf16_normal(rng, cap[r], Hkv, d) for r in range(R)] for _ in range(layers)]
    slab_start = np.concatenate([[0], np.cumsum(cap)]).astype(np.int64)
    dev_k = [cases.to_torch(np.concatenate(slabs_k[l]), True) for l in range(layers)]   # [sum cap, Hkv, d]
    dev_v = [cases.to_torch(np.concatenate(slabs_v[l]), True) for l in range(layers)]
    P = list(start)
    roots = np.array([5, 77], np.int32)
    total_accepted = 0
    for rnd in range(rounds):
        w = wl.small_workload(R=R, L=L, V=V, K=K, B=B, Hq=Hq, Hkv=Hkv, d=d, dtype="bf16", prefix_lens=tuple(P), index=90)
        logits = cases.drafter_batch(w, "peak", seed=100 + rnd)
        trees = [orc.build(logits[r], K, B, int(roots[r]), P[r]) for r in range(R)]
        tl = np.stack([wl.target_logits(w, trees[r].depth, r, "peak", seed=100 + rnd) for r in range(R)])
        q_h = bf16_normal(rng, layers, R, w.N, Hq, d)
        kt_h = bf16_normal(rng, layers, R, w.N, Hkv, d)
        vt_h = bf16_normal(rng, layers, R, w.N, Hkv, d)
        ks = rng.integers(0, 2 ** 32, (R, w.N), dtype=np.uint64)

        # ---- the round on the GPU -----------------------------------------------------------------
        tree = dd.ddtree_build(torch.from_numpy(logits).cuda(), K, B, torch.from_numpy(roots).cuda(),
                               torch.tensor(P, dtype=torch.int32).cuda())
        cu_host = np.concatenate([[0], np.cumsum(P)]).astype(np.int32)
        cu = torch.from_numpy(cu_host).cuda()
        outs = []
        for l in range(layers):
            # the attention call reads a packed cache: the requests' first P rows, back to back
            kc = torch.cat([dev_k[l][slab_start[r]:slab_start[r] + P[r]] for r in range(R)])
            vc = torch.cat([dev_v[l][slab_start[r]:slab_start[r] + P[r]] for r in range(R)])
            outs.append(dd.ddtree_tree_attention(cases.to_torch(q_h[l], True), kc, vc, cu_host.tolist(), cu,
                                                 cases.to_torch(kt_h[l], True), cases.to_torch(vt_h[l], True),
                                                 tree.anc_mask, tree.n_rows))
        t_dev = cases.to_torch(tl, True)
        if temperature > 0:
            acc = dd.ddtree_accept_sampled(t_dev, L, tree.node_token, tree.node_parent, tree.n_rows, temperature,
                                           torch.from_numpy(ks.astype(np.uint32).view(np.int32)).cuda())
        else:
            acc = dd.ddtree_accept(t_dev, L, tree.node_token, tree.node_parent, tree.n_rows)
        dst = torch.from_numpy(slab_start[:-1] + np.asarray(P, np.int64)).cuda()
        dd.ddtree_kv_compact([cases.to_torch(kt_h[l], True) for l in range(layers)],
                             [cases.to_torch(vt_h[l], True) for l in range(layers)], dev_k, dev_v, dst,
                             acc.accept_len, acc.accept_nodes)
        torch.cuda.synchronize()
        dd.device_status()

        # ---- the same round over the oracle, compared step by step ---------------------------------------
        new_roots = roots.copy()
        for r in range(R):
            ct = trees[r]
            cases.tree_arrays_equal(ct, tree, r)
            n = ct.n_rows
            x = wl.bf16_bits_to_f32(tl[r])
            choice = orc.node_sampled(x[:n], temperature, ks[r, :n]) if temperature > 0 else orc.node_argmax(x.astype(np.float64))[:n]
            walk = orc.accept_walk(ct.token, ct.parent, n, np.concatenate([choice, np.full(w.N - n, -1, np.int32)]))
            assert int(acc.accept_len[r]) == walk.accept_len and int(acc.bonus_token[r]) == walk.bonus_token, (rnd, r)
            assert list(acc.accept_nodes[r].cpu().numpy()[:walk.accept_len]) == walk.nodes
            assert list(acc.accept_tokens[r].cpu().numpy()[:walk.accept_len]) == walk.tokens
            for l in range(layers):
                ref, _ = orc.tree_attention(wl.bf16_to_f64(q_h[l, r]), wl.bf16_to_f64(slabs_k[l][r][:P[r]]),
                                            wl.bf16_to_f64(slabs_v[l][r][:P[r]]), wl.bf16_to_f64(kt_h[l, r]),
                                            wl.bf16_to_f64(vt_h[l, r]), ct.mask, n)
                got = outs[l][r, :n].float().cpu().numpy().astype(np.float64)
                err = np.abs(got - ref) / (1 + np.abs(ref))
                assert err.max() <= 1e-2, (rnd, r, l, err.max())
                # the oracle's cache after this round; the GPU's slab must hold the same bits
                slabs_k[l][r] = orc.kv_compact(slabs_k[l][r], kt_h[l, r], P[r], walk.nodes)
                slabs_v[l][r] = orc.kv_compact(slabs_v[l][r], vt_h[l, r], P[r], walk.nodes)
                for slab, dev_t in ((slabs_k[l][r], dev_k[l]), (slabs_v[l][r], dev_v[l])):
                    got_bits = dev_t[slab_start[r]:slab_start[r + 1]].view(torch.int16).cpu().numpy().view(np.uint16)
                    np.testing.assert_array_equal(got_bits, slab)
            new_roots[r] = walk.bonus_token
            P[r] += walk.accept_len + 1
            total_accepted += walk.accept_len
        roots = new_roots
    assert total_accepted >= 4  # the loop did move through accepted paths, not only bonus tokens
    assert all(P[r] <= cap[r] for r in range(R))
