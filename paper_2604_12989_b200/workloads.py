"""Seeded synthetic inputs for the DDTree per-round hot path.

This module only draws random numbers and shapes them; it holds none of the
method's arithmetic (no softmax, no tree search, no attention, no walk).  Both
the CPU oracle's tests and the CUDA path's tests/bench feed from it, so the two
sides always see identical arrays.

The paper evaluates on language-model benchmarks with trained drafter/target
checkpoints (Section 5.1, Appendix B); none of that is available offline, so the
tensors below only reproduce the *shapes and value distributions* of one
decoding round: a block of L drafter logit rows over a vocabulary of V tokens,
a KV-cache prefix plus one row of fresh K/V per tree node, and one target logit
row per tree node.

bf16 tensors are carried on the host as uint16 bit patterns (NumPy has no
bfloat16); `bf16_to_f64` converts them exactly.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

# --------------------------------------------------------------------------
# bf16 helpers (pure bit manipulation)
# --------------------------------------------------------------------------


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even), return uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp64."""
    return bf16_bits_to_f32(bits).astype(np.float64)


def round_through_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 -> fp32 (values land on the bf16 lattice, stored as fp32)."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


# --------------------------------------------------------------------------
# Workload table: the five configurations this build is measured on
# --------------------------------------------------------------------------


@dataclass(frozen=True)
class Workload:
    """Shapes of one synthetic decoding round.

    R requests; L block depth (draft positions after the bonus token); V
    vocabulary; K tokens kept per position; B node budget (root not counted,
    Section 4.2), so the verifier sees N = B + 1 rows.
    """

    index: int
    name: str
    R: int
    L: int
    V: int
    K: int
    B: int
    Hq: int
    Hkv: int
    d: int
    dtype: str  # "f32" or "bf16": element type of attention tensors and target logits
    prefix_lens: Tuple[int, ...]  # one per request
    layers: int
    noise: float  # std of the background logits
    boost0: float  # boost of the "true" token at depth 0
    boost_slope: float  # boost shrinks by this much per depth
    lattice: bool  # drafter logits pass through bf16 before being stored as fp32
    boost0_range: Optional[Tuple[float, float]] = None  # per-request U(lo, hi) instead of boost0

    @property
    def N(self) -> int:
        return self.B + 1

    @property
    def W(self) -> int:
        return (self.N + 31) // 32

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def cu_prefix(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.prefix_lens)]).astype(np.int32)


def _ragged_prefixes(seed: int, n: int, lo: int, hi: int) -> Tuple[int, ...]:
    rng = np.random.default_rng([seed, 3, 0, 99])
    return tuple(int(x) for x in rng.integers(lo, hi + 1, n))


def make_workloads(seed: int = 0) -> Dict[int, Workload]:
    return {
        0: Workload(0, "tiny", 1, 8, 1024, 4, 16, 4, 1, 64, "f32", (128,), 1, 2.0, 6.0, 0.5, False),
        1: Workload(1, "qwen3-8b-single", 1, 16, 151936, 8, 64, 32, 8, 128, "bf16", (4096,), 36, 3.0, 8.0, 0.4, True),
        2: Workload(2, "large-budget", 1, 16, 151936, 16, 256, 32, 8, 128, "bf16", (16384,), 36, 3.0, 8.0, 0.4, True),
        3: Workload(3, "ragged-batch", 16, 16, 151936, 8, 128, 32, 8, 128, "bf16",
                    _ragged_prefixes(seed, 16, 512, 8192), 36, 3.0, 8.0, 0.4, True, (3.0, 10.0)),
        4: Workload(4, "70b-long-context", 1, 16, 128256, 16, 512, 64, 8, 128, "bf16", (65536,), 80, 3.0, 8.0, 0.4, True),
    }


WORKLOADS = make_workloads(0)

VARIANTS = ("lit", "peak")
"""`lit`: boost added as written (b0 - c*depth).  `peak`: the same boost
multiplied by the noise std, which lifts the true token above the maximum of
~150k background draws so that drafted paths are actually accepted."""


def _rng(seed: int, cfg: int, request: int, stream: int, attempt: int = 0) -> np.random.Generator:
    return np.random.default_rng([seed, cfg, request, stream, attempt])


def small_workload(**kw) -> Workload:
    """An ad-hoc workload for tests (defaults = config 0)."""
    base = dict(index=9, name="adhoc", R=1, L=8, V=1024, K=4, B=16, Hq=4, Hkv=1, d=64, dtype="f32",
                prefix_lens=(128,), layers=1, noise=2.0, boost0=6.0, boost_slope=0.5, lattice=False)
    base.update(kw)
    if "prefix_lens" in kw:
        base["prefix_lens"] = tuple(int(p) for p in kw["prefix_lens"])
    return Workload(**base)


# --------------------------------------------------------------------------
# Drafter logits
# --------------------------------------------------------------------------

MIN_TOPK_GAP = 2e-3  # enforced fp32 gap between adjacent retained logits of one position
DITHER = 2.0 ** -5


def true_tokens(w: Workload, request: int, seed: int = 0) -> np.ndarray:
    """The seeded 'true' continuation y*_1..y*_{L+1} (one extra for the deepest target row)."""
    return _rng(seed, w.index, request, 0).integers(0, w.V, w.L + 1).astype(np.int32)


def request_boost0(w: Workload, request: int, seed: int = 0) -> float:
    if w.boost0_range is None:
        return w.boost0
    lo, hi = w.boost0_range
    return float(_rng(seed, w.index, request, 1).uniform(lo, hi))


def _boost(w: Workload, request: int, depth: np.ndarray, variant: str, seed: int) -> np.ndarray:
    b = request_boost0(w, request, seed) - w.boost_slope * depth
    if variant == "peak":
        b = b * w.noise
    elif variant != "lit":
        raise ValueError(f"unknown variant {variant!r}")
    return b.astype(np.float32)


def separate_top(row: np.ndarray, keep: int, rng: np.random.Generator) -> None:
    """Spread the `keep` largest entries of `row` (in place) so that adjacent ones
    differ by at least MIN_TOPK_GAP, and the last of them clears everything else
    by the same margin.  Entries are only ever raised, so which entries are the
    largest `keep` does not change.  Equal values are ordered by lower index."""
    V = row.shape[0]
    keep = min(keep, V)
    take = min(keep + 1, V)
    # indices of the `take` largest, ordered by (value desc, index asc)
    part = np.argpartition(-row, take - 1)[:take] if take < V else np.arange(V)
    thresh = row[part].min()
    cand = np.nonzero(row >= thresh)[0]
    order = cand[np.lexsort((cand, -row[cand]))][:take]
    top = order[:keep]
    row[top] = row[top] + rng.uniform(0.0, DITHER, keep).astype(np.float32)
    # re-sort the raised entries (dither may swap close ones), then push upwards
    top = top[np.lexsort((top, -row[top]))]
    floor = row[order[keep]] if take > keep else None
    for r in range(keep - 1, -1, -1):
        below = floor if r == keep - 1 else row[top[r + 1]]
        if below is not None:
            need = np.float32(below) + np.float32(MIN_TOPK_GAP)
            if row[top[r]] < need:
                row[top[r]] = need


def drafter_logits(w: Workload, request: int = 0, variant: str = "lit", seed: int = 0,
                   attempt: int = 0) -> np.ndarray:
    """fp32 [L, V] drafter logits for one request.

    Background ~ noise*N(0,1); at depth i (1-based) the true token y*_i gets
    +(boost0 - slope*i); optionally rounded through bf16; then the retained
    logits of every position are spread apart (see `separate_top`)."""
    rng = _rng(seed, w.index, request, 2, attempt)
    x = rng.standard_normal((w.L, w.V), dtype=np.float32) * np.float32(w.noise)
    y = true_tokens(w, request, seed)
    depth = np.arange(1, w.L + 1)
    x[np.arange(w.L), y[: w.L]] += _boost(w, request, depth, variant, seed)
    if w.lattice:
        x = round_through_bf16(x)
    drng = _rng(seed, w.index, request, 3, attempt)
    for i in range(w.L):
        separate_top(x[i], w.K, drng)
    return x


def drafter_logits_batch(w: Workload, variant: str = "lit", seed: int = 0,
                         attempts: Optional[List[int]] = None) -> np.ndarray:
    """fp32 [R, L, V]."""
    attempts = attempts or [0] * w.R
    return np.stack([drafter_logits(w, r, variant, seed, attempts[r]) for r in range(w.R)])


# --------------------------------------------------------------------------
# Target logits (one row per tree row; row i predicts the token after node i)
# --------------------------------------------------------------------------


def target_logits(w: Workload, node_depth: np.ndarray, request: int = 0, variant: str = "lit",
                  seed: int = 0) -> np.ndarray:
    """[N, V] target logits for one request: fp32 array, or uint16 bf16 bits when
    w.dtype == "bf16".  Row i sits at tree depth node_depth[i] (padding rows have
    depth -1 and get plain noise); it boosts the true token of the next position."""
    node_depth = np.asarray(node_depth)
    n = node_depth.shape[0]
    rng = _rng(seed, w.index, request, 4)
    y = true_tokens(w, request, seed)
    out_bits = np.empty((n, w.V), dtype=np.uint16) if w.dtype == "bf16" else None
    out = np.empty((n, w.V), dtype=np.float32) if w.dtype != "bf16" else None
    for i in range(n):
        row = rng.standard_normal(w.V, dtype=np.float32) * np.float32(w.noise)
        dpt = int(node_depth[i])
        if dpt >= 0:
            nxt = min(dpt + 1, w.L + 1)
            row[y[nxt - 1]] += _boost(w, request, np.array([nxt]), variant, seed)[0]
        if w.dtype == "bf16":
            out_bits[i] = f32_to_bf16_bits(row)
        else:
            out[i] = row
    return out_bits if w.dtype == "bf16" else out


# --------------------------------------------------------------------------
# Attention tensors
# --------------------------------------------------------------------------


@dataclass
class AttentionInputs:
    """One layer's tensors for all requests.  Arrays are fp32, or uint16 bf16
    bits when dtype == "bf16"."""

    q: np.ndarray  # [R, N, Hq, d]
    k_cache: np.ndarray  # [sum(P), Hkv, d]
    v_cache: np.ndarray
    k_tree: np.ndarray  # [R, N, Hkv, d]
    v_tree: np.ndarray
    cu_prefix: np.ndarray  # [R+1] int32
    dtype: str = "f32"
    extra: dict = field(default_factory=dict)

    def as_f64(self, name: str) -> np.ndarray:
        a = getattr(self, name)
        return bf16_to_f64(a) if self.dtype == "bf16" else a.astype(np.float64)


def attention_inputs(w: Workload, layer: int = 0, seed: int = 0) -> AttentionInputs:
    rng = _rng(seed, w.index, layer, 5)
    total_p = int(sum(w.prefix_lens))

    def draw(*shape):
        a = rng.standard_normal(shape, dtype=np.float32)
        return f32_to_bf16_bits(a) if w.dtype == "bf16" else a

    return AttentionInputs(
        q=draw(w.R, w.N, w.Hq, w.d),
        k_cache=draw(total_p, w.Hkv, w.d),
        v_cache=draw(total_p, w.Hkv, w.d),
        k_tree=draw(w.R, w.N, w.Hkv, w.d),
        v_tree=draw(w.R, w.N, w.Hkv, w.d),
        cu_prefix=w.cu_prefix,
        dtype=w.dtype,
    )


def root_tokens(w: Workload, seed: int = 0) -> np.ndarray:
    """[R] bonus token carried into the round (tree root)."""
    return _rng(seed, w.index, 0, 6).integers(0, w.V, w.R).astype(np.int32)
