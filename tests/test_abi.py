"""CPU-side checks of the C-ABI library: it loads, exports every symbol declared in
include/speca.h, and rejects bad arguments on the host before any CUDA call."""
import ctypes
import os
import re

import pytest

from paper_2607_16673_b200 import binding as speca
from paper_2607_16673_b200 import build as speca_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    speca_build.build()
    return speca.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "speca.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(speca_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert set(speca.EXPORTS) <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_version_and_strerror(lib):
    assert speca.version() == 100
    assert lib.speca_strerror(0) == b"ok"
    for code in range(-6, 0):
        assert lib.speca_strerror(code) not in (b"", b"ok", b"unknown speca error code")
    assert lib.speca_strerror(-99) == b"unknown speca error code"


def test_workspace_bytes_grows_with_nodes(lib):
    d = speca.Dims(24, 32, 16, 128, 256)
    a, b = speca.workspace_bytes(d, 0), speca.workspace_bytes(d, 4608)
    assert a > 0 and b > a and b < (1 << 22)


FAKE = ctypes.c_void_p(0x1000)        # aligned, never dereferenced: validation fails first
ODD = ctypes.c_void_p(0x1004)


def call_decode(lib, dims, ptrs=None):
    d = dims.c()
    ptrs = ptrs or [FAKE] * 7
    return lib.speca_decode_step(ctypes.byref(d), *ptrs, None)


def test_decode_rejects_bad_arguments_before_launch(lib):
    good = speca.Dims(1, 1, 4, 64, 64)
    assert call_decode(lib, good, [None] + [FAKE] * 6) == -1
    assert call_decode(lib, good, [ODD] + [FAKE] * 6) == -3
    assert call_decode(lib, speca.Dims(1, 1, 4, 96, 64)) == -2
    assert call_decode(lib, speca.Dims(1, 1, 4, 64, 48)) == -2
    assert call_decode(lib, speca.Dims(0, 1, 4, 64, 64)) == -4
    assert call_decode(lib, speca.Dims(1, 1, 4, 64, 64, max_depth=17)) == -4
    assert call_decode(lib, speca.Dims(1, 1, 4, 64, 64, max_nodes=0)) == -4
    assert call_decode(lib, speca.Dims(1, 1, 4, 64, 64, route=7)) == -2
    assert lib.speca_decode_step(None, *([FAKE] * 7), None) == -1


def test_verify_and_commit_reject_bad_arguments_before_launch(lib):
    dims = speca.Dims(1, 2, 4, 64, 64, max_nodes=8)
    d = dims.c()
    need = speca.workspace_bytes(dims, 8)
    args = [FAKE] * 7 + [8, FAKE, FAKE, FAKE, None, FAKE, need, FAKE, None]
    # a complete argument list with total_nodes == 0 is accepted without launching anything
    zero = list(args); zero[7] = 0
    assert lib.speca_verify_tree(ctypes.byref(d), *zero) == 0
    bad = list(args); bad[13] = need - 1
    assert lib.speca_verify_tree(ctypes.byref(d), *bad) == -6
    bad = list(args); bad[12] = None
    assert lib.speca_verify_tree(ctypes.byref(d), *bad) == -6
    bad = list(args); bad[8] = None                    # parent
    assert lib.speca_verify_tree(ctypes.byref(d), *bad) == -1
    bad = list(args); bad[7] = 17                      # more nodes than batch * max_nodes
    assert lib.speca_verify_tree(ctypes.byref(d), *bad) == -4
    bad = list(args); bad[7] = -1
    assert lib.speca_verify_tree(ctypes.byref(d), *bad) == -4
    bad = list(args); bad[10] = ODD                    # o misaligned
    assert lib.speca_verify_tree(ctypes.byref(d), *bad) == -3
    cargs = [FAKE] * 6 + [0, None, FAKE, FAKE, FAKE, None]
    assert lib.speca_commit(ctypes.byref(d), *cargs) == 0
    bad = list(cargs); bad[0] = None
    assert lib.speca_commit(ctypes.byref(d), *bad) == -1
    bad = list(cargs); bad[6] = -3
    assert lib.speca_commit(ctypes.byref(d), *bad) == -4
    assert lib.speca_greedy_accept(0, 8, *([FAKE] * 9), None) == -4
    assert lib.speca_greedy_accept(2, 8, None, *([FAKE] * 8), None) == -1


def test_binding_refuses_to_run_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(speca, "_lib", None)
    monkeypatch.setattr(speca, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(speca.SpecaError):
        speca.version()
