"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

import paper_2608_12629_b200 as cake
from paper_2608_12629_b200 import build as cake_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def library():
    cake_build.build_library()
    return ctypes.CDLL(cake.LIB_PATH)


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "cake_kmeans.h")).read()
    return sorted(set(re.findall(r"CAKE_API\s+[\w\s\*]+?\b(cake_\w+)\s*\(", text)))


def test_header_declares_the_three_named_calls():
    names = declared_symbols()
    for n in ("cake_kmeans_assign", "cake_kmeans_update", "cake_kmeans_lloyd"):
        assert n in names


def test_library_exports_every_declared_symbol(library):
    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(library, n), f"{n} declared in the header but not exported"
    assert sorted(names) == sorted(cake.EXPORTS), "binding and header disagree on the entry points"


def test_host_only_calls(library):
    assert cake.cake_version() >= 100
    assert cake.strerror(cake.CAKE_OK) == "ok"
    assert "workspace" in cake.strerror(cake.CAKE_ERR_WORKSPACE)
    assert cake.strerror(12345).startswith("unknown")
    small = cake.cake_kmeans_workspace_bytes(1, 1000, 64, 16)
    big = cake.cake_kmeans_workspace_bytes(1, 100000, 64, 16)
    assert 0 < small < big and small % 256 == 0
    assert cake.cake_kmeans_workspace_bytes(4, 1000, 64, 16) < cake.cake_kmeans_workspace_bytes(8, 1000, 64, 16)
    assert cake.cake_kmeans_lloyd_host_device_bytes(1, 1000, 64, 16, 3) > small
    for bad in [(0, 10, 8, 2), (1, -1, 8, 2), (1, 10, 0, 2), (1, 10, 8, 0)]:
        with pytest.raises(cake.CakeError) as e:
            cake.cake_kmeans_workspace_bytes(*bad)
        assert e.value.code == cake.CAKE_ERR_SHAPE


def test_argument_checks_need_no_device(library):
    sz = ctypes.c_size_t(0)
    assert library.cake_kmeans_workspace_bytes(ctypes.c_longlong(1), ctypes.c_longlong(8), 8, 2, None) == cake.CAKE_ERR_NULL
    # null workspace / null centroids are rejected before any CUDA call
    L = cake.lib()
    rc = L.cake_kmeans_assign(None, None, 8, 8, 2, None, None, None, 0, None, 0)
    assert rc == cake.CAKE_ERR_NULL
    rc = L.cake_kmeans_lloyd(None, None, 8, 8, 2, -1, None, None, None, None, None, None, None, 0, None, 0)
    assert rc == cake.CAKE_ERR_SHAPE
