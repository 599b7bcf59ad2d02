"""Host-side checks that need no GPU: the C-ABI library builds, loads, and exports every
symbol the header declares; size/layout queries and host arithmetic behave."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2601_07396_b200 import binding as sc
from paper_2601_07396_b200 import build as sc_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "svdcache.h")


@pytest.fixture(scope="module")
def lib():
    sc_build.build()
    return sc.lib()


def _declared():
    text = open(HEADER).read()
    return re.findall(r"SVDCACHE_API\s+[\w\s\*]+?\b(svdcache_\w+)\s*\(", text)


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = _declared()
    assert len(names) >= 20 and len(set(names)) == len(names)
    raw = ctypes.CDLL(sc.LIB_PATH)
    for n in names:
        assert getattr(raw, n) is not None
    assert set(names) == set(sc.SIGNATURES), set(names) ^ set(sc.SIGNATURES)
    # the python layer keeps the same names
    for n in names:
        if n not in ("svdcache_status_string", "svdcache_last_cuda_error"):
            assert hasattr(sc, n), n


def test_status_strings(lib):
    assert lib.svdcache_status_string(0) == b"ok"
    for code in range(-8, 0):
        assert lib.svdcache_status_string(code) not in (b"", b"unknown status")
    assert lib.svdcache_status_string(-99) == b"unknown status"


def test_layout_queries_are_consistent(lib):
    for (N, D, k, dt) in [(256, 1152, 32, sc.F32), (4608, 3072, 64, sc.BF16), (118800, 3072, 128, sc.BF16),
                          (1, 8, 8, sc.F32)]:
        eb = 4 if dt == sc.F32 else 2
        co, ro = sc.svdcache_state_layout(N, D, k, dt)
        total = sc.svdcache_state_bytes(N, D, k, dt)
        assert co == 256 and ro % 256 == 0 and ro >= co + N * k * 4
        assert total % 256 == 0 and total >= ro + N * D * eb
        a, b, c, d = sc.svdcache_basis_layout(D, k, dt)
        tb = sc.svdcache_basis_bytes(D, k, dt)
        assert a == 256 and b >= a + D * k * 4 and all(x % 256 == 0 for x in (a, b, c, d))
        if dt == sc.BF16:
            assert c >= b + D * k * 4 and d >= c + D * k * 2 and tb >= d + D * k * 2
        else:
            assert tb >= b + D * k * 4
        assert sc.svdcache_calibrate_workspace_bytes(D, k) >= D * D * 8


def test_shape_limits_are_enforced_on_the_host(lib):
    out = ctypes.c_size_t(0)
    assert lib.svdcache_state_bytes(0, 64, 8, 0, ctypes.byref(out)) == -2
    assert lib.svdcache_state_bytes(10, 60, 8, 0, ctypes.byref(out)) == -2     # D % 8
    assert lib.svdcache_state_bytes(10, 64, 12, 0, ctypes.byref(out)) == -2    # k % 8
    assert lib.svdcache_state_bytes(10, 64, 128, 0, ctypes.byref(out)) == -2   # k > D
    assert lib.svdcache_state_bytes(10, 512, 264, 0, ctypes.byref(out)) == -2  # k > 256
    assert lib.svdcache_state_bytes(10, 64, 8, 7, ctypes.byref(out)) == -1     # dtype
    assert lib.svdcache_state_bytes(10, 64, 8, 0, None) == -1
    assert lib.svdcache_set_path(9) == -1


def test_rank_for_energy_is_eq6(lib):
    lam = [8.0, 4.0, 2.0, 1.0, 1.0]
    assert sc.svdcache_rank_for_energy(lam, 16.0, 0.5) == 1
    assert sc.svdcache_rank_for_energy(lam, 16.0, 0.51) == 2
    assert sc.svdcache_rank_for_energy(lam, 16.0, 0.85) == 3
    assert sc.svdcache_rank_for_energy(lam, 16.0, 1.0) == 5
    assert sc.svdcache_rank_for_energy(lam[:2], 16.0, 0.99) == 2
    # same rule as the oracle on a random spectrum
    from oracle import svdcache_oracle as oracle
    rng = np.random.default_rng(0)
    lam = np.sort(rng.uniform(0, 1, 40))[::-1]
    for tau in (0.3, 0.6, 0.85, 0.95):
        assert sc.svdcache_rank_for_energy(lam, lam.sum() * 1.1, tau) == \
            oracle.rank_for_energy(lam, lam.sum() * 1.1, tau)
    out = ctypes.c_int(0)
    assert lib.svdcache_rank_for_energy(None, 3, 1.0, 0.5, ctypes.byref(out)) == -1


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2601_07396_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle|svdcache_oracle|liboracle", text, re.M), \
                    f"{f} reaches into the oracle"
