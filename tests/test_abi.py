"""The C-ABI library builds, loads and exports every symbol include/ab.h declares; host-side
argument checks reject bad calls before anything is launched.  No GPU needed."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2405_01067_b200 import build
    build.build()
    from paper_2405_01067_b200 import binding
    return binding.lib()


def test_every_declared_symbol_is_exported(L):
    hdr = open(os.path.join(ROOT, "include", "ab.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(ab_[a-z0-9_]+)\s*\(", hdr))
    assert {"ab_layer_forward", "ab_layer_backward", "ab_group_average", "ab_recombine", "ab_svd_split"} <= names
    for nm in names:
        assert hasattr(L, nm), nm
    from paper_2405_01067_b200 import binding
    assert set(binding.EXPORTS) <= names


def test_status_strings(L):
    from paper_2405_01067_b200 import binding as b
    assert b.status_string(0) == "ok"
    for code in range(-7, 0):
        assert b.status_string(code) not in ("ok", "unknown status")
    assert b.status_string(-99) == "unknown status"
    assert L.ab_version().decode().count(".") == 1


def test_workspace_query(L):
    from paper_2405_01067_b200 import binding as b
    assert b.ab_workspace_bytes(b.AB_OP_LAYER_FORWARD, 64, 256, 512, 32) >= 64 * 32 * 4
    assert b.ab_workspace_bytes(b.AB_OP_LAYER_BACKWARD, 64, 256, 512, 32) >= 2 * 64 * 32 * 4
    assert b.ab_workspace_bytes(b.AB_OP_SVD_SPLIT, 0, 256, 512, 32) >= 2 * 256 * 256 * 4
    assert b.ab_workspace_bytes(b.AB_OP_SVD_SPLIT, 0, 0, 512, 32) == 0
    assert b.ab_workspace_bytes(99, 1, 1, 1, 1) == 0


def test_host_side_rejections(L):
    from paper_2405_01067_b200 import binding as b
    p = ctypes.c_void_p(256)          # never dereferenced: every call below fails its checks first
    bad = b.AB_ERR_INVALID_ARG
    # NULL pointers, non-positive sizes, r beyond min(m,n), short leading dimensions, unknown dtype
    assert L.ab_layer_forward(None, p, p, p, None, 4, 8, 8, 2, 2, 8, 0, p, 1024, None) == bad
    assert L.ab_layer_forward(p, p, p, None, None, 4, 8, 8, 2, 2, 8, 0, p, 1024, None) == bad
    assert L.ab_layer_forward(p, p, p, p, None, 4, 0, 8, 2, 2, 8, 0, p, 1024, None) == bad
    assert L.ab_layer_forward(p, p, p, p, None, 4, 8, 8, 9, 9, 8, 0, p, 1024, None) == bad
    assert L.ab_layer_forward(p, p, p, p, None, 4, 8, 8, 2, 1, 8, 0, p, 1024, None) == bad
    assert L.ab_layer_forward(p, p, p, p, None, 4, 8, 8, 2, 2, 7, 0, p, 1024, None) == bad
    assert L.ab_layer_forward(p, p, p, p, None, 4, 8, 8, 2, 2, 8, 5, p, 1024, None) == bad
    assert L.ab_layer_forward(p, p, p, p, None, -1, 8, 8, 2, 2, 8, 0, p, 1024, None) == bad
    assert L.ab_layer_backward(p, None, p, p, None, p, None, None, 4, 8, 8, 2, 2, 8, 0, p, 1024, None) == bad
    assert L.ab_group_average(p, 16, 0, 16, 0, 0, p, None) == bad
    assert L.ab_group_average(p, 8, 2, 16, 0, 0, p, None) == bad       # overlapping copies
    assert L.ab_group_average(None, 16, 2, 16, 0, 0, p, None) == bad
    assert L.ab_group_average(p, 16, 65, 16, 0, 0, p, None) == b.AB_ERR_UNSUPPORTED
    assert L.ab_recombine(p, p, None, 4, 4, 2, 2, 4, 0, None, 0, None) == bad
    assert L.ab_recombine(p, p, p, 4, 4, 2, 1, 4, 0, None, 0, None) == bad
    assert L.ab_svd_split(p, 4, 4, 0, 0.0, p, p, p, p, p, 0, 0, p, 1 << 20, None) == bad
    assert L.ab_svd_split(p, 4, 4, 2, -1.0, p, p, p, p, p, 0, 0, p, 1 << 20, None) == bad
    assert L.ab_svd_split(p, 4, 4, 2, float("nan"), p, p, p, p, p, 0, 0, p, 1 << 20, None) == bad
    assert L.ab_svd_split(p, 4000, 4000, 2, 0.0, p, p, p, p, p, 0, 0, p, 1 << 20, None) == b.AB_ERR_UNSUPPORTED
    assert L.ab_svd_split(p, 4, 4, 2, 0.0, p, p, p, p, p, 0, 0, None, 0, None) == b.AB_ERR_WORKSPACE
    assert L.ab_svd_split(p, 4, 4, 2, 0.0, p, p, p, p, p, 0, 0, ctypes.c_void_p(264), 1 << 20, None) == b.AB_ERR_WORKSPACE
    assert L.ab_group_sync(None, 1, 2, 0.1, 0, None, p, 1024, None, 0) == bad


def test_no_device_means_an_error_not_a_fallback(L):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    from paper_2405_01067_b200 import binding as b
    p = ctypes.c_void_p(256)
    assert L.ab_group_average(p, 16, 2, 16, 0, 0, p, None) == b.AB_ERR_CUDA
    assert L.ab_recombine(p, p, p, 4, 4, 2, 2, 4, 0, None, 0, None) == b.AB_ERR_CUDA
    assert L.ab_layer_forward(p, p, p, p, None, 4, 8, 8, 2, 2, 8, 0, p, 1024, None) == b.AB_ERR_CUDA


def test_package_never_imports_the_checker():
    pkg = os.path.join(ROOT, "paper_2405_01067_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f


def test_static_forward_rejects_sizes_that_would_wrap(L):
    """N * r is checked by division: a row count near 2^63 (or 2^58 at r = 64, whose product wraps to a
    small number) is refused on the host, before any launch, with or without a device."""
    from paper_2405_01067_b200 import binding as b
    p = ctypes.c_void_p(256)
    for N in ((2 ** 63 - 1) // 2, 2 ** 58, 2 ** 58 + 1):
        assert L.ab_layer_forward_static(p, p, p, p, N, 128, 128, 64, 64, 128, 0, None) == b.AB_ERR_UNSUPPORTED
