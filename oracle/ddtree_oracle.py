"""CPU oracle for the DDTree per-round hot path (test infrastructure only).

A plain, slow, fp64 NumPy restatement of what one DDTree decoding round
computes between the drafter's logits and the next bonus token.  It exists to
check the CUDA library; it is NOT part of the product: only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may import it, and it shares no
code with the CUDA path.  Every function names the passage of the paper it
follows.  All functions are pinned by tests against closed forms, brute force
or library routines; the order in which Algorithm 1 pops equal or nearly equal
scores is not part of any contract ("ties broken arbitrarily", Proposition 2)
and is therefore exposed only for diagnostics.

Notation follows the paper: L draft positions, vocabulary V, rank tuples
rho = (rho_1..rho_d) with 1-based ranks, sigma(rho) = sum_i log q_i^(rho_i),
node budget B (the root -- the bonus token b -- is not counted, Section 4.2).
"""
from __future__ import annotations

import heapq
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

# --------------------------------------------------------------------------
# Section 3: per-position distributions  q_i = softmax(l_i)
# --------------------------------------------------------------------------


def log_softmax(logits: np.ndarray) -> np.ndarray:
    """log q_i(v) = l_i(v) - log sum_v' exp l_i(v'), row-wise over the last axis,
    in fp64 (Section 3: q_i = softmax(l_i); Section 4.3 works with log q)."""
    x = np.asarray(logits, dtype=np.float64)
    m = x.max(axis=-1, keepdims=True)
    lse = m + np.log(np.exp(x - m).sum(axis=-1, keepdims=True))
    return x - lse


def top_k(logits: np.ndarray, K: int) -> Tuple[np.ndarray, np.ndarray]:
    """Per position i the K most probable tokens v_i^(1..K) and log q_i^(k)
    (Section 4.3, the ordering q_i(v^(1)) >= q_i(v^(2)) >= ...).

    Softmax is monotone, so tokens are ordered on the raw logits, which makes
    the order exact; equal logits are ordered by lower token id.
    Returns (tok [L,K] int64, lq [L,K] float64)."""
    x = np.asarray(logits, dtype=np.float64)
    L, V = x.shape
    if not 1 <= K <= V:
        raise ValueError("need 1 <= K <= V")
    lq_full = log_softmax(x)
    ids = np.arange(V)
    tok = np.empty((L, K), dtype=np.int64)
    lq = np.empty((L, K), dtype=np.float64)
    for i in range(L):
        order = np.lexsort((ids, -x[i]))  # primary key: logit descending; secondary: id ascending
        tok[i] = order[:K]
        lq[i] = lq_full[i, order[:K]]
    return tok, lq


# --------------------------------------------------------------------------
# Algorithm 1: best-first construction
# --------------------------------------------------------------------------


@dataclass
class PoppedNode:
    rho: Tuple[int, ...]  # 1-based ranks, one per depth
    sigma: float


def best_first_tree(lq: np.ndarray, B: int) -> Tuple[List[PoppedNode], Optional[float]]:
    """Algorithm 1.  `lq[i-1][k-1]` = log q_i^(k) for depth i and rank k.

    Max-heap keyed by sigma, started with the tuple (1).  While fewer than B
    tuples are popped and the heap is non-empty: pop the best tuple rho of depth
    d, add it to T; if rho_d + 1 <= K push the next sibling with score
    sigma - log q_d^(rho_d) + log q_d^(rho_d + 1); if d < L push the first child
    with score sigma + log q_{d+1}^(1).

    Equal scores pop shallower-first, then lexicographically smaller rho (only to
    make this function deterministic).  Returns the popped nodes in pop order and
    the best score left in the heap (None if it ran empty)."""
    lq = np.asarray(lq, dtype=np.float64)
    L, K = lq.shape
    heap: list = []
    heapq.heappush(heap, (-lq[0, 0], 1, (1,)))
    T: List[PoppedNode] = []
    while len(T) < B and heap:
        neg, d, rho = heapq.heappop(heap)
        sigma = -neg
        T.append(PoppedNode(rho, sigma))
        r = rho[-1]
        if r + 1 <= K:
            s_sib = sigma - lq[d - 1, r - 1] + lq[d - 1, r]
            heapq.heappush(heap, (-s_sib, d, rho[:-1] + (r + 1,)))
        if d < L:
            s_child = sigma + lq[d, 0]
            heapq.heappush(heap, (-s_child, d + 1, rho + (1,)))
    left = -heap[0][0] if heap else None
    return T, left


def boundary_gap(lq: np.ndarray, B: int) -> float:
    """sigma of the B-th popped tuple minus the best score left behind; +inf when
    the heap ran empty.  A positive gap means the top-B set is unique
    (Proposition 2's "ties broken arbitrarily" does not bite)."""
    T, left = best_first_tree(lq, B)
    if left is None or len(T) < B:
        return float("inf")
    return T[-1].sigma - left


# --------------------------------------------------------------------------
# Section 4.4: compile the tree for the verifier
# --------------------------------------------------------------------------


@dataclass
class CompiledTree:
    n_rows: int  # 1 + number of nodes
    token: np.ndarray  # [B+1] int32, row 0 = bonus token b; padding -1
    parent: np.ndarray  # [B+1] int32, row 0 = -1; padding -1
    depth: np.ndarray  # [B+1] int32, row 0 = 0; padding -1
    position_ids: np.ndarray  # [B+1] int32 = prefix_len + depth; padding -1
    mask: np.ndarray  # [B+1, W] uint32 ancestor-or-self bits, LSB = column 0
    first_child: np.ndarray  # [B+1] int32 (-1 if none)
    child_count: np.ndarray  # [B+1] int32
    logprob: np.ndarray  # [B+1] float64 sigma per row (root 0)
    rho: List[Tuple[int, ...]]  # rank tuple per row (root = ())


def compile_tree(nodes: Sequence[PoppedNode], tok: np.ndarray, root_token: int, prefix_len: int,
                 B: int) -> CompiledTree:
    """Flatten the tree into the verifier's inputs (Section 4.4): a sequence of
    token ids rooted at b, position ids by tree depth, and the mask under which a
    node sees the root, its ancestors and itself.

    The paper leaves the flattening order open.  Here rows are in level order:
    sorted by (depth, rank tuple), which depends only on the node *set*, puts
    every parent before its children and keeps siblings adjacent in rank order.
    The bonus token sits at absolute position prefix_len (it is not in the KV
    cache yet, Section 3), so position_ids = prefix_len + depth."""
    N = B + 1
    W = (N + 31) // 32
    rhos = sorted((n.rho for n in nodes), key=lambda r: (len(r), r))
    sig = {n.rho: n.sigma for n in nodes}
    row_of = {(): 0}
    for i, r in enumerate(rhos):
        row_of[r] = i + 1
    n_rows = len(rhos) + 1
    token = np.full(N, -1, np.int32)
    parent = np.full(N, -1, np.int32)
    depth = np.full(N, -1, np.int32)
    pos = np.full(N, -1, np.int32)
    mask = np.zeros((N, W), np.uint32)
    first_child = np.full(N, -1, np.int32)
    child_count = np.zeros(N, np.int32)
    logprob = np.zeros(N, np.float64)
    token[0], depth[0], pos[0] = root_token, 0, prefix_len
    mask[0, 0] = 1
    for r in rhos:
        i = row_of[r]
        d = len(r)
        p = row_of[r[:-1]]  # prefix-closed: the parent tuple is in the tree
        token[i] = tok[d - 1, r[-1] - 1]
        parent[i] = p
        depth[i] = d
        pos[i] = prefix_len + d
        mask[i] = mask[p]
        mask[i, i // 32] |= np.uint32(1) << np.uint32(i % 32)
        logprob[i] = sig[r]
        if first_child[p] < 0:
            first_child[p] = i
        child_count[p] += 1
    return CompiledTree(n_rows, token, parent, depth, pos, mask, first_child, child_count, logprob,
                        [()] + rhos)


def build(drafter_logits: np.ndarray, K: int, B: int, root_token: int, prefix_len: int) -> CompiledTree:
    """Steps 2-3 of the round (Section 4.1) for one request: [L,V] logits ->
    compiled draft tree."""
    tok, lq = top_k(drafter_logits, K)
    nodes, _ = best_first_tree(lq, B)
    return compile_tree(nodes, tok, root_token, prefix_len, B)


# --------------------------------------------------------------------------
# Section 4.4: tree attention in the verifier
# --------------------------------------------------------------------------


def visible(mask: np.ndarray, n_rows: int) -> np.ndarray:
    """Boolean [n_rows, n_rows]: vis[i, j] = bit j of mask row i."""
    cols = np.arange(n_rows)
    words = mask[:n_rows][:, cols // 32]
    return ((words >> (cols % 32).astype(np.uint32)) & 1).astype(bool)


def tree_attention(q: np.ndarray, k_prefix: np.ndarray, v_prefix: np.ndarray, k_tree: np.ndarray,
                   v_tree: np.ndarray, mask: np.ndarray, n_rows: int, scale: Optional[float] = None,
                   rows: Optional[Sequence[int]] = None, heads: Optional[Sequence[int]] = None
                   ) -> Tuple[np.ndarray, np.ndarray]:
    """Tree attention for one request and one layer (Section 4.4): row i attends to
    every key of the KV-cache prefix and, inside the tree, only to the rows whose
    bit is set in mask[i] (root, ancestors, itself).

    q [N,Hq,d]; k_prefix/v_prefix [P,Hkv,d]; k_tree/v_tree [N,Hkv,d]; all fp64.
    Query head h uses KV head h // (Hq // Hkv).  scale defaults to 1/sqrt(d)
    (the default of the scaled-dot-product attention the paper uses, App. B).
    Returns (out [len(rows), len(heads), d], lse [len(rows), len(heads)]);
    `rows`/`heads` default to all rows < n_rows and all heads."""
    q = np.asarray(q, np.float64)
    N, Hq, d = q.shape
    Hkv = k_tree.shape[1]
    G = Hq // Hkv
    P = k_prefix.shape[0]
    scale = 1.0 / np.sqrt(d) if not scale else scale
    rows = list(range(n_rows)) if rows is None else list(rows)
    heads = list(range(Hq)) if heads is None else list(heads)
    vis = visible(mask, n_rows)
    out = np.zeros((len(rows), len(heads), d))
    lse = np.zeros((len(rows), len(heads)))
    for hi, h in enumerate(heads):
        kv = h // G
        keys = np.concatenate([k_prefix[:, kv], k_tree[:n_rows, kv]], axis=0).astype(np.float64)
        vals = np.concatenate([v_prefix[:, kv], v_tree[:n_rows, kv]], axis=0).astype(np.float64)
        for ri, i in enumerate(rows):
            see = np.concatenate([np.ones(P, bool), vis[i]])
            s = (keys[see] @ q[i, h]) * scale
            m = s.max()
            p = np.exp(s - m)
            z = p.sum()
            out[ri, hi] = (p / z) @ vals[see]
            lse[ri, hi] = m + np.log(z)
    return out, lse


# --------------------------------------------------------------------------
# Section 4.4: verification walk (greedy decoding rule)
# --------------------------------------------------------------------------


def node_argmax(target_logits: np.ndarray) -> np.ndarray:
    """The target's greedy choice at every row: the smallest token id attaining the
    row maximum (Section 4.4: the target's own decoding rule, greedy case)."""
    x = np.asarray(target_logits, np.float64)
    return np.argmax(x, axis=-1).astype(np.int32)  # numpy returns the first maximum


@dataclass
class Acceptance:
    accept_len: int  # accepted drafted nodes (the bonus token is not counted)
    nodes: List[int]  # rows of the accepted path, in order
    tokens: List[int]
    bonus_token: int  # first unmatched target token = next round's root


def accept_walk(token: np.ndarray, parent: np.ndarray, n_rows: int, choice: np.ndarray) -> Acceptance:
    """Verifier walk (Section 4.4, Figure 2(b)): start at the root; while the
    target's choice at the current row equals the token of one of its children,
    accept that child and move there; otherwise stop.  The target's choice at the
    last accepted row is the next bonus token."""
    cur = 0
    path: List[int] = []
    while True:
        want = int(choice[cur])
        nxt = -1
        for j in range(n_rows):
            if parent[j] == cur and token[j] == want:
                nxt = j
                break
        if nxt < 0:
            break
        path.append(nxt)
        cur = nxt
    return Acceptance(len(path), path, [int(token[j]) for j in path], int(choice[cur]))


# --------------------------------------------------------------------------
# Section 4.4: verification walk (temperature-based sampling rule)
# --------------------------------------------------------------------------
#
# Section 4.4 lets the verification follow whichever rule the target decodes by,
# greedy or sampling at a temperature: at temperature T > 0 the target's choice at a
# row is a token drawn from softmax(t / T).  The paper does not say how the draw
# is made.  For the draw to be a function of its inputs that two programs can
# agree on bit for bit, it is defined here as an inverse-CDF draw in token order
# over fixed-point weights:
#   * the random input is one 32-bit integer k per row, u = k / 2^32;
#   * weight of token v: W_v = floor(2^40 * e_v) with e_v = 2^((x_v - max x) * c),
#     c = float32(log2(e) / float32(T)), evaluated in float32 with one rounding per operation:
#     t = (x_v - max) * c; n = t rounded to the nearest integer (ties to even: what adding and subtracting
#     1.5 * 2^23 in float32 does); f = t - n, in [-1/2, 1/2]; p(f) = a degree-5 polynomial for 2^f in Horner
#     form (multiply, then add), a float32 in [0.707, 1.415]; e_v = p(f) * 2^n taken apart into the 24-bit
#     significand of p and a shift, so that no rounding happens after p; tokens with t < -40 get 0;
#   * the draw is the smallest v whose inclusive prefix sum of W exceeds floor(total * k / 2^32).
# Integer sums do not depend on the order of summation, so a parallel program gets the same token.
# The weights differ from the numerators of softmax(t / T) by less than 5e-6 relative (pinned in the tests).

SAMPLING_POLY = (np.float32(0.693147004), np.float32(0.240222424), np.float32(0.0555073358),
                 np.float32(0.00967151299), np.float32(0.00132647273))  # coefficients of f^1 .. f^5
_ROUND_MAGIC = np.float32(12582912.0)  # 1.5 * 2^23: float32 addition rounds to an integer in [2^23, 2^24)


def sampling_weights(row: np.ndarray, temperature: float) -> List[int]:
    """Fixed-point weights W_v of one row of target logits at temperature T (see above)."""
    f32 = np.float32
    x = np.asarray(row, f32)
    c = f32(1.4426950408889634 / float(f32(temperature)))  # the temperature crosses the C boundary as a float32
    with np.errstate(invalid="ignore", over="ignore"):
        t = ((x - x.max()).astype(f32) * c).astype(f32)    # float32 subtract, float32 multiply
        live = t >= f32(-40.0)                             # false for -inf and NaN too
        t = np.where(live, t, f32(0.0)).astype(f32)
        r = (t + _ROUND_MAGIC).astype(f32)
        n = r.view(np.uint32).astype(np.int64) - 0x4B400000
        f = (t - (r - _ROUND_MAGIC).astype(f32)).astype(f32)
        acc = np.full_like(f, SAMPLING_POLY[4])
        for k in (3, 2, 1, 0):
            acc = (acc * f).astype(f32)
            acc = (acc + SAMPLING_POLY[k]).astype(f32)
        acc = (acc * f).astype(f32)
        acc = (acc + f32(1.0)).astype(f32)
    bits = acc.view(np.uint32).astype(np.int64)
    sig = (bits & 0x7FFFFF) | 0x800000                     # p = sig * 2^(e - 23)
    e = (bits >> 23) - 127
    out: List[int] = []
    for ok, s_, e_, n_ in zip(live.tolist(), sig.tolist(), e.tolist(), n.tolist()):
        if not ok:
            out.append(0)
            continue
        sh = e_ + 17 + n_                                  # floor(p * 2^n * 2^40) = sig * 2^(e - 23 + n + 40)
        out.append(s_ << sh if sh >= 0 else s_ >> -sh)
    return out


def sample_token(row: np.ndarray, temperature: float, k: int) -> int:
    """The target's choice at one row under temperature sampling with random input k in [0, 2^32)."""
    w = sampling_weights(row, temperature)
    total = sum(w)
    thr = (total * int(k)) >> 32
    acc = 0
    for v, wv in enumerate(w):
        acc += wv
        if acc > thr:
            return v
    raise ValueError("row without a finite maximum")


def node_sampled(target_logits: np.ndarray, temperature: float, uniforms: np.ndarray) -> np.ndarray:
    """The target's sampled choice at every row ([rows, V] logits, one 32-bit integer per row)."""
    return np.array([sample_token(target_logits[i], temperature, int(uniforms[i]))
                     for i in range(target_logits.shape[0])], np.int32)


# --------------------------------------------------------------------------
# Section 4.4: position ids by tree depth, consumed by the verifier's positional encoding
# --------------------------------------------------------------------------


def rope(x: np.ndarray, positions: np.ndarray, theta: float) -> np.ndarray:
    """Rotary positional encoding of the rows of x ([rows, heads, d], d even) at the given integer
    positions (Section 4.4 assigns position ids by tree depth so that every node is encoded at the position
    it would have in its own branch; the target models of the paper, Qwen3, use rotary embeddings in the
    half-split form).  Pair (j, j + d/2) of every head is rotated by the angle
    positions[row] * theta^(-2j/d): as complex numbers z_j = x_j + i x_{j+d/2}, out = z_j * exp(i * angle)."""
    x = np.asarray(x, np.float64)
    rows, heads, d = x.shape
    half = d // 2
    inv_freq = float(theta) ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    ang = np.asarray(positions, np.float64)[:, None] * inv_freq[None, :]
    z = (x[..., :half] + 1j * x[..., half:]) * np.exp(1j * ang)[:, None, :]
    return np.concatenate([z.real, z.imag], axis=-1)


def kv_compact(cache: np.ndarray, tree_rows: np.ndarray, prefix_len: int, path: Sequence[int]) -> np.ndarray:
    """End of a round (Section 4.4: after the walk only the accepted path stays in
    the cache): the keys (or values) of the root and of the accepted nodes are
    appended to the cached context in path order, i.e. the root lands at cache
    position prefix_len and the i-th accepted node at prefix_len + i, which is
    the position id it was verified at (its depth).  `cache` is [rows, ...] with
    at least prefix_len + len(path) + 1 rows; returns the updated copy."""
    out = cache.copy()
    out[prefix_len] = tree_rows[0]
    for i, j in enumerate(path):
        out[prefix_len + 1 + i] = tree_rows[j]
    return out
