"""Python binding of the DDTree B200 library (libddtree.so, C ABI in include/ddtree.h).

The functions here only marshal arguments: they take torch CUDA tensors (device memory and
streams are PyTorch's), allocate outputs and workspaces, and pass raw pointers to the three
entry points.  Every step of the round runs in the library's kernels; there is no fallback:
if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libddtree.so")

DDTREE_F32, DDTREE_BF16 = 0, 1

EXPORTS = (
    "ddtree_status_string", "ddtree_last_error",
    "ddtree_build_workspace_bytes", "ddtree_build",
    "ddtree_tree_attention_workspace_bytes", "ddtree_tree_attention", "ddtree_tree_attention_rope",
    "ddtree_accept_workspace_bytes", "ddtree_accept", "ddtree_accept_static_scratch",
    "ddtree_accept_sampled_workspace_bytes", "ddtree_accept_sampled",
    "ddtree_kv_compact", "ddtree_rope_tree",
    "ddtree_device_status", "ddtree_selftest_wait_timeout", "ddtree_tree_attention_set_path", "ddtree_tree_attention_kernel_count",
)

_lib = None


class DDTreeError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"ddtree status {status}: {message}")
        self.status = status


def lib() -> ctypes.CDLL:
    """Load libddtree.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2604_12989_b200._build` "
                               "(or __graft_entry__.build()); there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        c = ctypes
        vp, i32, i64, sz, f32 = c.c_void_p, c.c_int, c.c_int64, c.c_size_t, c.c_float
        L.ddtree_status_string.restype = c.c_char_p
        L.ddtree_status_string.argtypes = [i32]
        L.ddtree_last_error.restype = c.c_char_p
        L.ddtree_last_error.argtypes = []
        L.ddtree_build_workspace_bytes.restype = sz
        L.ddtree_build_workspace_bytes.argtypes = [i32] * 5
        L.ddtree_build.restype = i32
        L.ddtree_build.argtypes = [vp, i32, i64, i32, i32, i32, i32, i32] + [vp] * 13 + [vp, sz, vp]
        L.ddtree_tree_attention_workspace_bytes.restype = sz
        L.ddtree_tree_attention_workspace_bytes.argtypes = [i32] * 6 + [vp]
        L.ddtree_tree_attention.restype = i32
        L.ddtree_tree_attention.argtypes = [vp] * 11 + [i32] * 6 + [f32, vp, sz, vp]
        L.ddtree_tree_attention_rope.restype = i32
        L.ddtree_tree_attention_rope.argtypes = [vp] * 10 + [f32, vp, vp] + [i32] * 6 + [f32, vp, sz, vp]
        L.ddtree_accept_workspace_bytes.restype = sz
        L.ddtree_accept_workspace_bytes.argtypes = [i32] * 3
        L.ddtree_accept.restype = i32
        L.ddtree_accept.argtypes = [vp, i32, i64, i32, i32, i32, i32] + [vp] * 8 + [vp, sz, vp]
        L.ddtree_accept_static_scratch.restype = i32
        L.ddtree_accept_static_scratch.argtypes = [vp, i32, i64, i32, i32, i32, i32] + [vp] * 8 + [vp]
        L.ddtree_accept_sampled_workspace_bytes.restype = sz
        L.ddtree_accept_sampled_workspace_bytes.argtypes = [i32] * 3
        L.ddtree_accept_sampled.restype = i32
        L.ddtree_accept_sampled.argtypes = [vp, i32, i64, i32, i32, i32, i32] + [vp] * 3 + [f32, vp] + [vp] * 5 + [vp, sz, vp]
        L.ddtree_rope_tree.restype = i32
        L.ddtree_rope_tree.argtypes = [vp, vp, vp, vp] + [i32] * 6 + [f32, vp]
        L.ddtree_kv_compact.restype = i32
        L.ddtree_kv_compact.argtypes = [i32] * 7 + [vp] * 7 + [vp]
        L.ddtree_device_status.restype = i32
        L.ddtree_device_status.argtypes = []
        L.ddtree_tree_attention_kernel_count.restype = i32
        L.ddtree_tree_attention_kernel_count.argtypes = [i32] * 6 + [vp]
        L.ddtree_tree_attention_set_path.restype = i32
        L.ddtree_tree_attention_set_path.argtypes = [i32]
        L.ddtree_selftest_wait_timeout.restype = i32
        L.ddtree_selftest_wait_timeout.argtypes = [vp]
        _lib = L
    return _lib


def _check(rc: int) -> None:
    if rc != 0:
        raise DDTreeError(rc, lib().ddtree_last_error().decode())


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return DDTREE_F32
    if t.dtype == torch.bfloat16:
        return DDTREE_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _stream(stream=None) -> int:
    import torch
    return (stream or torch.cuda.current_stream()).cuda_stream


def _scratch(nbytes: int, device, stream=None):
    """A temporary workspace for one call.  The kernels are only enqueued when the call returns, so the block
    must not go back to the caching allocator's pool of another stream while they run: when the call is made on a
    stream that is not the current one, the block is tied to that stream."""
    import torch
    t = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    if stream is not None and stream != torch.cuda.current_stream(device):
        t.record_stream(stream)
    return t


@dataclass
class Tree:
    """Outputs of ddtree_build (torch CUDA tensors).  Shapes: [R] or [R, B+1(, W)]."""
    n_rows: "torch.Tensor"
    node_token: "torch.Tensor"
    node_parent: "torch.Tensor"
    node_depth: "torch.Tensor"
    position_ids: "torch.Tensor"
    anc_mask: "torch.Tensor"  # int32 storage of the uint32 words
    first_child: "torch.Tensor"
    child_count: "torch.Tensor"
    node_logprob: "torch.Tensor"
    topk_token: "torch.Tensor"
    topk_logprob: "torch.Tensor"
    B: int
    L: int
    K: int


def ddtree_build(drafter_logits, K: int, B: int, root_token, prefix_len, workspace=None, out: Optional[Tree] = None,
                 stream=None) -> Tree:
    """drafter_logits [R, L, V] (fp32 or bf16, CUDA, last dim contiguous); root_token, prefix_len [R] int32."""
    import torch
    R, L, V = drafter_logits.shape
    assert drafter_logits.is_cuda and drafter_logits.stride(2) == 1
    assert R == 1 or drafter_logits.stride(0) == L * drafter_logits.stride(1)
    dev = drafter_logits.device
    N, W = B + 1, (B + 1 + 31) // 32
    if out is None:
        i32 = dict(dtype=torch.int32, device=dev)
        out = Tree(torch.empty(R, **i32), torch.empty(R, N, **i32), torch.empty(R, N, **i32), torch.empty(R, N, **i32),
                   torch.empty(R, N, **i32), torch.empty(R, N, W, **i32), torch.empty(R, N, **i32),
                   torch.empty(R, N, **i32), torch.empty(R, N, dtype=torch.float32, device=dev),
                   torch.empty(R, L, K, **i32), torch.empty(R, L, K, dtype=torch.float32, device=dev), B, L, K)
    need = lib().ddtree_build_workspace_bytes(R, L, V, K, B)
    if workspace is None:
        workspace = _scratch(need, dev, stream)
    _check(lib().ddtree_build(
        drafter_logits.data_ptr(), _dtype_code(drafter_logits), drafter_logits.stride(1), R, L, V, K, B,
        root_token.data_ptr(), prefix_len.data_ptr(), out.n_rows.data_ptr(), out.node_token.data_ptr(),
        out.node_parent.data_ptr(), out.node_depth.data_ptr(), out.position_ids.data_ptr(), out.anc_mask.data_ptr(),
        _ptr(out.first_child), _ptr(out.child_count), _ptr(out.node_logprob), _ptr(out.topk_token),
        _ptr(out.topk_logprob), workspace.data_ptr(), workspace.numel(), _stream(stream)))
    return out


def tree_attention_workspace_bytes(R, B, Hq, Hkv, d, dtype_code, cu_prefix_host) -> int:
    arr = (ctypes.c_int32 * (R + 1))(*[int(x) for x in cu_prefix_host])
    return lib().ddtree_tree_attention_workspace_bytes(R, B, Hq, Hkv, d, dtype_code, ctypes.addressof(arr))


def tree_attention_kernel_count(R, B, Hq, Hkv, d, dtype_code, cu_prefix_host) -> int:
    """Kernels one ddtree_tree_attention call with these shapes launches (1, or 2 with a split merge)."""
    arr = (ctypes.c_int32 * (R + 1))(*[int(x) for x in cu_prefix_host])
    return lib().ddtree_tree_attention_kernel_count(R, B, Hq, Hkv, d, dtype_code, ctypes.addressof(arr))


def ddtree_tree_attention(q, k_cache, v_cache, cu_prefix_host, cu_prefix, k_tree, v_tree, anc_mask, n_rows,
                          out=None, lse=None, softmax_scale: float = 0.0, workspace=None, stream=None):
    """q [R, B+1, Hq, d]; k_cache/v_cache [sum P, Hkv, d]; k_tree/v_tree [R, B+1, Hkv, d];
    cu_prefix_host: sequence of R+1 ints (host); cu_prefix: int32 CUDA tensor with the same values.
    Returns `out` ([R, B+1, Hq, d], same dtype as q; padding rows untouched)."""
    import torch
    R, N, Hq, d = q.shape
    Hkv = k_tree.shape[2]
    B = N - 1
    for t in (q, k_cache, v_cache, k_tree, v_tree):
        assert t.is_cuda and t.is_contiguous() and t.dtype == q.dtype
    if out is None:
        out = torch.zeros_like(q)
    code = _dtype_code(q)
    arr = (ctypes.c_int32 * (R + 1))(*[int(x) for x in cu_prefix_host])
    if workspace is None:
        need = lib().ddtree_tree_attention_workspace_bytes(R, B, Hq, Hkv, d, code, ctypes.addressof(arr))
        workspace = _scratch(need, q.device, stream)
    _check(lib().ddtree_tree_attention(
        q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), ctypes.addressof(arr), cu_prefix.data_ptr(),
        k_tree.data_ptr(), v_tree.data_ptr(), anc_mask.data_ptr(), n_rows.data_ptr(), out.data_ptr(), _ptr(lse),
        code, R, B, Hq, Hkv, d, float(softmax_scale), workspace.data_ptr(), workspace.numel(), _stream(stream)))
    return out


def ddtree_tree_attention_rope(q, k_cache, v_cache, cu_prefix_host, cu_prefix, k_tree, v_tree, anc_mask, n_rows,
                               position_ids, rope_theta: float, out=None, lse=None, softmax_scale: float = 0.0,
                               workspace=None, stream=None):
    """ddtree_tree_attention on UNROTATED bf16 q / k_tree: the rotary encoding at `position_ids` ([R, B+1], as
    written by ddtree_build) is applied inside the kernel; q and k_tree are left as they are."""
    import torch
    R, N, Hq, d = q.shape
    Hkv = k_tree.shape[2]
    B = N - 1
    for t in (q, k_cache, v_cache, k_tree, v_tree):
        assert t.is_cuda and t.is_contiguous() and t.dtype == q.dtype
    if out is None:
        out = torch.zeros_like(q)
    code = _dtype_code(q)
    arr = (ctypes.c_int32 * (R + 1))(*[int(x) for x in cu_prefix_host])
    if workspace is None:
        need = lib().ddtree_tree_attention_workspace_bytes(R, B, Hq, Hkv, d, code, ctypes.addressof(arr))
        workspace = _scratch(need, q.device, stream)
    _check(lib().ddtree_tree_attention_rope(
        q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), ctypes.addressof(arr), cu_prefix.data_ptr(),
        k_tree.data_ptr(), v_tree.data_ptr(), anc_mask.data_ptr(), n_rows.data_ptr(), position_ids.data_ptr(),
        float(rope_theta), out.data_ptr(), _ptr(lse), code, R, B, Hq, Hkv, d, float(softmax_scale),
        workspace.data_ptr(), workspace.numel(), _stream(stream)))
    return out


@dataclass
class Acceptance:
    accept_len: "torch.Tensor"  # [R]
    accept_nodes: "torch.Tensor"  # [R, L]
    accept_tokens: "torch.Tensor"  # [R, L]
    bonus_token: "torch.Tensor"  # [R]
    node_argmax: "torch.Tensor"  # [R, B+1]


def ddtree_accept(target_logits, L: int, node_token, node_parent, n_rows, workspace=None,
                  out: Optional[Acceptance] = None, stream=None) -> Acceptance:
    """target_logits [R, B+1, V] (fp32 or bf16, CUDA)."""
    import torch
    R, N, V = target_logits.shape
    B = N - 1
    assert target_logits.is_cuda and target_logits.stride(2) == 1
    assert R == 1 or target_logits.stride(0) == N * target_logits.stride(1)
    dev = target_logits.device
    if out is None:
        i32 = dict(dtype=torch.int32, device=dev)
        out = Acceptance(torch.empty(R, **i32), torch.empty(R, L, **i32), torch.empty(R, L, **i32),
                         torch.empty(R, **i32), torch.empty(R, N, **i32))
    if workspace is None:
        workspace = _scratch(lib().ddtree_accept_workspace_bytes(R, B, V), dev, stream)
    _check(lib().ddtree_accept(
        target_logits.data_ptr(), _dtype_code(target_logits), target_logits.stride(1), R, B, V, L,
        node_token.data_ptr(), node_parent.data_ptr(), n_rows.data_ptr(), out.accept_len.data_ptr(),
        out.accept_nodes.data_ptr(), out.accept_tokens.data_ptr(), out.bonus_token.data_ptr(),
        _ptr(out.node_argmax), workspace.data_ptr(), workspace.numel(), _stream(stream)))
    return out


def ddtree_accept_sampled(target_logits, L: int, node_token, node_parent, n_rows, temperature: float, row_uniform,
                          workspace=None, out: Optional[Acceptance] = None, stream=None, all_rows: bool = True) -> Acceptance:
    """ddtree_accept under the temperature-based decoding rule: the target's choice at a row is drawn from
    softmax(target_logits / temperature) with the row's 32-bit random input (row_uniform: [R, B+1], an int32
    or uint32 CUDA tensor whose bit patterns are used).  `node_argmax` of the result holds the drawn tokens of
    every row; with all_rows=False the call draws only at the rows the walk stands on (much cheaper) and leaves
    `node_argmax` untouched."""
    import torch
    R, N, V = target_logits.shape
    B = N - 1
    assert target_logits.is_cuda and target_logits.stride(2) == 1
    assert R == 1 or target_logits.stride(0) == N * target_logits.stride(1)
    assert row_uniform.is_cuda and row_uniform.is_contiguous() and row_uniform.numel() == R * N and row_uniform.element_size() == 4
    dev = target_logits.device
    if out is None:
        i32 = dict(dtype=torch.int32, device=dev)
        out = Acceptance(torch.empty(R, **i32), torch.empty(R, L, **i32), torch.empty(R, L, **i32),
                         torch.empty(R, **i32), torch.empty(R, N, **i32))
    if workspace is None:
        workspace = _scratch(lib().ddtree_accept_sampled_workspace_bytes(R, B, V), dev, stream)
    _check(lib().ddtree_accept_sampled(
        target_logits.data_ptr(), _dtype_code(target_logits), target_logits.stride(1), R, B, V, L,
        node_token.data_ptr(), node_parent.data_ptr(), n_rows.data_ptr(), float(temperature), row_uniform.data_ptr(),
        out.accept_len.data_ptr(), out.accept_nodes.data_ptr(), out.accept_tokens.data_ptr(), out.bonus_token.data_ptr(),
        _ptr(out.node_argmax) if all_rows else None, workspace.data_ptr(), workspace.numel(), _stream(stream)))
    return out


STATIC_SCRATCH_BYTES = 256 * 1024


def ddtree_accept_static_scratch(target_logits, L: int, node_token, node_parent, n_rows, out: Acceptance,
                                 stream=None) -> Acceptance:
    """ddtree_accept for callers that cannot provide a workspace: the per-chunk partials go to a
    fixed array inside the library (STATIC_SCRATCH_BYTES per GPU).  This wrapper allocates nothing
    either: `out` must be given.  Calls on one device share the array, so do not let two of them
    overlap on the GPU; make the first call on a device outside any stream capture."""
    R, N, V = target_logits.shape
    assert target_logits.is_cuda and target_logits.stride(2) == 1
    assert R == 1 or target_logits.stride(0) == N * target_logits.stride(1)
    _check(lib().ddtree_accept_static_scratch(
        target_logits.data_ptr(), _dtype_code(target_logits), target_logits.stride(1), R, N - 1, V, L,
        node_token.data_ptr(), node_parent.data_ptr(), n_rows.data_ptr(), out.accept_len.data_ptr(),
        out.accept_nodes.data_ptr(), out.accept_tokens.data_ptr(), out.bonus_token.data_ptr(),
        _ptr(out.node_argmax), _stream(stream)))
    return out


def ddtree_rope_tree(q, k_tree, position_ids, n_rows, rope_theta: float, stream=None) -> None:
    """Rotary positional encoding, in place, of the tree's query rows q [R, B+1, Hq, d] and key rows k_tree
    [R, B+1, Hkv, d] (either may be None) at the position ids written by ddtree_build."""
    t = q if q is not None else k_tree
    assert t is not None and t.is_cuda and t.is_contiguous()
    R, N, _, d = t.shape
    Hq = q.shape[2] if q is not None else 1
    Hkv = k_tree.shape[2] if k_tree is not None else 1
    for u in (q, k_tree):
        assert u is None or (u.is_cuda and u.is_contiguous() and u.dtype == t.dtype and u.shape[0] == R and u.shape[1] == N and u.shape[3] == d)
    _check(lib().ddtree_rope_tree(_ptr(q), _ptr(k_tree), position_ids.data_ptr(), n_rows.data_ptr(), _dtype_code(t),
                                  R, N - 1, Hq, Hkv, d, float(rope_theta), _stream(stream)))


def ddtree_kv_compact(k_tree, v_tree, k_cache, v_cache, dst_row, accept_len, accept_nodes, stream=None) -> None:
    """End of a round: copy the root's and the accepted nodes' K/V rows of every layer to cache rows
    dst_row[r], dst_row[r]+1, ...  k_tree / v_tree: lists (one entry per layer) of [R, B+1, Hkv, d]
    tensors; k_cache / v_cache: lists of [rows, Hkv, d] tensors, updated in place; dst_row: int64 [R];
    accept_len, accept_nodes: as returned by ddtree_accept."""
    import ctypes as c
    layers = len(k_tree)
    assert layers >= 1 and len(v_tree) == layers and len(k_cache) == layers and len(v_cache) == layers
    R, N, Hkv, d = k_tree[0].shape
    L = accept_nodes.shape[1]
    for t in list(k_tree) + list(v_tree):
        assert t.is_cuda and t.is_contiguous() and tuple(t.shape) == (R, N, Hkv, d) and t.dtype == k_tree[0].dtype
    for t in list(k_cache) + list(v_cache):
        assert t.is_cuda and t.is_contiguous() and tuple(t.shape[1:]) == (Hkv, d) and t.dtype == k_tree[0].dtype
    import torch
    assert dst_row.dtype == torch.int64 and dst_row.is_cuda and dst_row.numel() == R
    arr = lambda ts: (c.c_void_p * layers)(*[t.data_ptr() for t in ts])
    _check(lib().ddtree_kv_compact(R, N - 1, L, Hkv, d, _dtype_code(k_tree[0]), layers, arr(k_tree), arr(v_tree),
                                   arr(k_cache), arr(v_cache), dst_row.data_ptr(), accept_len.data_ptr(),
                                   accept_nodes.data_ptr(), _stream(stream)))


def tree_attention_set_path(path: int) -> None:
    """0: the library chooses the bf16 attention kernel per call; 1 / 2: force the two-row-tile / one-row-tile kernel."""
    _check(lib().ddtree_tree_attention_set_path(int(path)))


def selftest_wait_timeout(stream=None) -> None:
    """Enqueue the library's one-thread kernel whose bounded wait runs out (see include/ddtree.h); the next
    device_status() raises DDTreeError with status 5 (device-side wait timed out), the one after passes."""
    _check(lib().ddtree_selftest_wait_timeout(_stream(stream)))


def device_status() -> None:
    """Synchronise and raise if a bounded device-side wait gave up since the last call."""
    _check(lib().ddtree_device_status())
