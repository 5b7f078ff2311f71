"""CPU-only checks of the boundary: the shared library builds, loads without a GPU and exports
every symbol include/ddtree.h declares; argument validation answers without launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2604_12989_b200 import _build
    import paper_2604_12989_b200 as dd
    _build.build()
    return dd.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ddtree.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ddtree_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    import paper_2604_12989_b200 as dd
    names = declared_symbols()
    assert len(names) >= 9
    for n in names:
        assert hasattr(lib, n), n
    assert set(dd.EXPORTS) == set(names)


def test_status_strings(lib):
    assert lib.ddtree_status_string(0) == b"ok"
    assert b"workspace" in lib.ddtree_status_string(3)


def test_workspace_queries(lib):
    assert lib.ddtree_build_workspace_bytes(1, 16, 151936, 8, 64) > 0
    assert lib.ddtree_build_workspace_bytes(1, 16, 151936, 64, 64) == 0  # K > 32
    assert lib.ddtree_accept_workspace_bytes(16, 128, 151936) > 0
    cu = (ctypes.c_int32 * 2)(0, 4096)
    assert lib.ddtree_tree_attention_workspace_bytes(1, 64, 32, 8, 128, 1, ctypes.addressof(cu)) > 0
    assert lib.ddtree_tree_attention_workspace_bytes(1, 64, 32, 7, 128, 1, ctypes.addressof(cu)) == 0


def test_validation_without_gpu(lib):
    none = [None] * 13
    assert lib.ddtree_build(None, 0, 0, 1, 1, 1, 1, 1, *none, None, 0, None) == 1
    assert b"logits is NULL" in lib.ddtree_last_error()
    buf = ctypes.create_string_buffer(4096)
    p = (ctypes.addressof(buf) + 15) & ~15
    assert lib.ddtree_build(p, 0, 8, 1, 1, 8, 9, 1, *none, None, 0, None) == 1  # K > V
    assert lib.ddtree_build(p, 7, 8, 1, 1, 8, 2, 1, *none, None, 0, None) == 1  # bad dtype
    assert lib.ddtree_build(p + 4, 0, 8, 1, 1, 8, 2, 1, *none, None, 0, None) == 1  # misaligned
    assert lib.ddtree_accept(p, 0, 8, 1, 1, 8, 1, *([None] * 8), None, 0, None) == 1  # null outputs
    # ddtree_kv_compact: every refusal happens on the host, before any launch
    ptrs = (ctypes.c_void_p * 2)(p, p)
    assert lib.ddtree_kv_compact(1, 8, 4, 2, 64, 1, 2, None, ptrs, ptrs, ptrs, p, p, p, None) == 1       # NULL table
    assert lib.ddtree_kv_compact(1, 8, 4, 1, 4, 1, 2, ptrs, ptrs, ptrs, ptrs, p, p, p, None) == 2        # 8-byte rows
    assert b"multiple of 16" in lib.ddtree_last_error()
    bad = (ctypes.c_void_p * 2)(p, p + 4)
    assert lib.ddtree_kv_compact(1, 8, 4, 2, 64, 1, 2, ptrs, bad, ptrs, ptrs, p, p, p, None) == 1        # misaligned layer buffer
    assert lib.ddtree_kv_compact(1, 8, 4, 2, 64, 9, 2, ptrs, ptrs, ptrs, ptrs, p, p, p, None) == 1       # bad dtype
    assert lib.ddtree_kv_compact(1, 8, 4, 2, 64, 1, 0, ptrs, ptrs, ptrs, ptrs, p, p, p, None) == 1       # no layers
    # ddtree_accept_sampled: temperature and pointers are checked on the host
    sampled = lambda T, u=p: lib.ddtree_accept_sampled(p, 0, 8, 1, 1, 8, 1, p, p, p, T, u, p, p, p, p, None, p, 1 << 20, None)
    assert sampled(0.0) == 1 and b"temperature" in lib.ddtree_last_error()
    assert sampled(-2.0) == 1
    assert sampled(float("inf")) == 1
    assert sampled(float("nan")) == 1
    assert sampled(1.0, None) == 1 and b"NULL" in lib.ddtree_last_error()                                # no random inputs
    assert lib.ddtree_accept_sampled(p, 0, 8, 1, 1, 8, 1, p, p, p, 1.0, p, p, p, p, p, None, p, 16, None) == 3  # workspace too small
    assert lib.ddtree_accept_sampled_workspace_bytes(1, 64, 151936) > lib.ddtree_accept_workspace_bytes(1, 64, 151936)
    assert lib.ddtree_accept_sampled_workspace_bytes(1, 4096, 151936) == 0                               # B out of range
    # ddtree_rope_tree
    rope = lambda d=128, theta=1e6, q=p, k=p, dt=1: lib.ddtree_rope_tree(q, k, p, p, dt, 1, 8, 4, 2, d, theta, None)
    assert rope(d=7) == 2 and b"head_dim" in lib.ddtree_last_error()      # odd head dimension
    assert rope(d=512) == 2
    assert rope(theta=0.0) == 1 and rope(theta=float("inf")) == 1
    assert rope(q=None, k=None) == 1
    assert rope(dt=5) == 1
    assert lib.ddtree_rope_tree(p, p, None, p, 1, 1, 8, 4, 2, 128, 1e6, None) == 1   # no position ids


def test_attention_kernel_choice_hook(lib):
    """ddtree_tree_attention_set_path takes 0, 1 or 2 and refuses anything else; the workspace query does not
    depend on it (it covers every kernel the call may pick)."""
    cu = (ctypes.c_int32 * 2)(0, 4096)
    sizes = []
    for path in (0, 1, 2, 0):
        assert lib.ddtree_tree_attention_set_path(path) == 0
        sizes.append(lib.ddtree_tree_attention_workspace_bytes(1, 64, 32, 8, 128, 1, cu))
    assert len(set(sizes)) == 1 and sizes[0] > 0
    for bad in (-1, 3, 100):
        assert lib.ddtree_tree_attention_set_path(bad) == 1
    assert b"path" in lib.ddtree_last_error()


def test_attention_kernel_count(lib):
    """One kernel when the rows fill the GPU (no KV split), two when a single request's KV range is split; fp32: one."""
    lib.ddtree_tree_attention_set_path(0)
    one = (ctypes.c_int32 * 2)(0, 4096)
    assert lib.ddtree_tree_attention_kernel_count(1, 64, 32, 8, 128, 1, one) == 2
    assert lib.ddtree_tree_attention_kernel_count(1, 16, 4, 1, 64, 0, one) == 1
    many = (ctypes.c_int32 * 65)(*[512 * i for i in range(65)])
    assert lib.ddtree_tree_attention_kernel_count(64, 128, 32, 8, 128, 1, many) == 1
    assert lib.ddtree_tree_attention_kernel_count(1, 64, 32, 7, 128, 1, one) == 0  # Hq not a multiple of Hkv
