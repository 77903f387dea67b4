"""The C-ABI library loads and exports every symbol the public header declares; host-side argument
checks answer before anything is launched.  Runs without a GPU (no compute calls)."""
import ctypes
import os
import re

import pytest

from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import build as tbn_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    tbn_build.build()
    return B.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "tbn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tbn_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_symbols()
    assert "tbn_linear_fwd" in names and "tbn_conv2d_fwd" in names and "tbn_mlp_fwd" in names
    assert "tbn_aggregate_tile" in names and "tbn_pack_tile" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in tbn.h but not exported"
        assert n in B.SIGNATURES, f"{n} has no ctypes signature in the binding"
    assert sorted(B.SIGNATURES) == names


def test_tile_words(lib):
    assert [lib.tbn_tile_words(q) for q in (0, 1, 32, 33, 128, 129, 65536)] == [0, 4, 4, 4, 4, 8, 2048]


def test_status_strings(lib):
    seen = {lib.tbn_status_string(s) for s in range(-6, 1)}
    assert len(seen) == 7 and all(seen)


def test_argument_errors_are_found_on_the_host(lib):
    dummy = 0x1000   # never dereferenced: every call below must fail validation first
    args = [dummy, B.BF16, 4, 64, 64, dummy, 4, dummy, B.ALPHA_PER_TILE, None, B.ACT_NONE, dummy, B.BF16,
            None, 0, None]
    bad = list(args); bad[0] = None
    assert lib.tbn_linear_fwd(*bad) == -1                     # null x
    bad = list(args); bad[6] = 3
    assert lib.tbn_linear_fwd(*bad) == -2                     # k does not divide N
    bad = list(args); bad[1] = 7
    assert lib.tbn_linear_fwd(*bad) == -1                     # unknown dtype
    bad = list(args); bad[0] = dummy + 2
    assert lib.tbn_linear_fwd(*bad) == -1                     # misaligned x
    bad = list(args); bad[2] = -1
    assert lib.tbn_linear_fwd(*bad) == -1                     # negative T
    assert lib.tbn_linear_fwd_path(*(args + [9])) == -1       # unknown path
    assert lib.tbn_aggregate_tile(dummy, None, 10, 3, 0, dummy, dummy, dummy, 1 << 20, None) == -2
    assert lib.tbn_aggregate_tile(dummy, None, 12, 3, 0, dummy, dummy, None, 0, None) == -4
    assert lib.tbn_pack_tile(None, 8, dummy, None) == -1
    # the scratch-free variant refuses layers beyond its built-in 1 MiB array (it needs about N/512 bytes)
    assert lib.tbn_aggregate_tile_static(dummy, None, 1 << 31, 2, 0, dummy, dummy, None) == -4
    assert lib.tbn_aggregate_tile_static(dummy, None, 10, 3, 0, dummy, dummy, None) == -2
    # the exact limit: q = 1 needs 16 + 8 k bytes, so k = 131071 (and the k = N = 131072 case) no longer fit
    assert lib.tbn_aggregate_tile_static(dummy, None, 131071, 131071, 1, dummy, dummy, None) == -4
    assert lib.tbn_aggregate_tile_static(dummy, None, 131072, 131072, 1, dummy, dummy, None) == -4
    assert lib.tbn_linear_select_path(4, 64, 64, 3, B.BF16) == -2
    conv = [dummy, B.BF16, 1, 3, 8, 8, 4, 3, 3, 1, 1, dummy, 5, dummy, 0, None, 0, dummy, B.BF16, None, 0, None]
    assert lib.tbn_conv2d_fwd(*conv) == -2                    # 108 weights, k = 5
    conv[8] = 30
    assert lib.tbn_conv2d_fwd(*conv) == -2                    # filter larger than padded input


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/libtbn.so")
    with pytest.raises(RuntimeError):
        B.lib()
