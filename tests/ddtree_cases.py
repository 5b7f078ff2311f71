"""Test-side glue: draws a workload, runs the CPU oracle on it and moves the same arrays to the
GPU.  Imports both the oracle and the input generators; the CUDA binding is imported lazily by
the GPU tests only."""
from __future__ import annotations

import functools
from typing import List

import numpy as np

from oracle import ddtree_oracle as orc
from paper_2604_12989_b200 import workloads as wl

MIN_BOUNDARY_GAP = 1e-3


@functools.lru_cache(maxsize=None)
def accepted_attempt(w: wl.Workload, request: int, variant: str, seed: int = 0) -> int:
    """First redraw of the drafter logits whose top-B prefix set is separated from the rest by
    at least MIN_BOUNDARY_GAP in log-probability, so that fp32 rounding cannot change the set."""
    for attempt in range(64):
        x = wl.drafter_logits(w, request, variant, seed, attempt)
        _, lq = orc.top_k(x, w.K)
        if orc.boundary_gap(lq, w.B) >= MIN_BOUNDARY_GAP:
            return attempt
    raise RuntimeError("no separated draw found")


def drafter_batch(w: wl.Workload, variant: str, seed: int = 0) -> np.ndarray:
    attempts = [accepted_attempt(w, r, variant, seed) for r in range(w.R)]
    return wl.drafter_logits_batch(w, variant, seed, attempts)


def oracle_trees(w: wl.Workload, logits: np.ndarray, roots: np.ndarray) -> List[orc.CompiledTree]:
    return [orc.build(logits[r], w.K, w.B, int(roots[r]), int(w.prefix_lens[r])) for r in range(w.R)]


def to_f64(w: wl.Workload, a: np.ndarray) -> np.ndarray:
    return wl.bf16_to_f64(a) if w.dtype == "bf16" else a.astype(np.float64)


def to_torch(a: np.ndarray, bf16: bool = False, device="cuda"):
    import torch
    if bf16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


def tree_arrays_equal(ct: orc.CompiledTree, tree, r: int) -> None:
    """Bit-exact comparison of one request's tree arrays (GPU `tree` vs oracle `ct`)."""
    n = int(tree.n_rows[r].item())
    assert n == ct.n_rows
    for name, want in (("node_token", ct.token), ("node_parent", ct.parent), ("node_depth", ct.depth),
                       ("position_ids", ct.position_ids), ("first_child", ct.first_child),
                       ("child_count", ct.child_count)):
        got = getattr(tree, name)[r].cpu().numpy()
        np.testing.assert_array_equal(got, want, err_msg=name)
    got_mask = tree.anc_mask[r].cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(got_mask, ct.mask, err_msg="anc_mask")
    np.testing.assert_allclose(tree.node_logprob[r].cpu().numpy(), ct.logprob, atol=2e-4, rtol=0)


class Guard:
    """CUDA tensors between two poisoned margins.  The GPU tests hand every output and workspace of a call
    to the library in such a tensor and check afterwards that the margins still hold the poison: a kernel
    that writes outside the buffer it was given is caught without a memory checker."""

    MARGIN = 4096  # bytes on either side (keeps the 256-byte alignment of the payload)
    POISON = 0xA5

    def __init__(self):
        self.items = []

    def empty(self, shape, dtype, fill=None):
        import torch
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        buf = torch.full((2 * self.MARGIN + (n + 255) // 256 * 256,), self.POISON, dtype=torch.uint8, device="cuda")
        view = buf[self.MARGIN:self.MARGIN + n].view(dtype).view(*shape)
        if fill is not None:
            view.fill_(fill)
        self.items.append((buf, n))
        return view

    def check(self):
        import torch
        torch.cuda.synchronize()
        for k, (buf, n) in enumerate(self.items):
            assert bool((buf[:self.MARGIN] == self.POISON).all()), f"buffer {k}: bytes before it were overwritten"
            assert bool((buf[self.MARGIN + n:] == self.POISON).all()), f"buffer {k}: bytes behind it were overwritten"


def guarded_tree(g: Guard, R: int, L: int, K: int, B: int):
    """A Tree (outputs of ddtree_build) whose every array sits between guard bands."""
    import torch
    import paper_2604_12989_b200 as dd
    N, W = B + 1, (B + 1 + 31) // 32
    i32, f32 = torch.int32, torch.float32
    return dd.Tree(g.empty((R,), i32), g.empty((R, N), i32), g.empty((R, N), i32), g.empty((R, N), i32),
                   g.empty((R, N), i32), g.empty((R, N, W), i32), g.empty((R, N), i32), g.empty((R, N), i32),
                   g.empty((R, N), f32), g.empty((R, L, K), i32), g.empty((R, L, K), f32), B, L, K)


def guarded_acceptance(g: Guard, R: int, L: int, N: int):
    import torch
    import paper_2604_12989_b200 as dd
    i32 = torch.int32
    return dd.Acceptance(g.empty((R,), i32), g.empty((R, L), i32), g.empty((R, L), i32), g.empty((R,), i32),
                         g.empty((R, N), i32))
