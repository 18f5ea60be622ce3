"""The C-ABI library builds for sm_100a, loads without a GPU, and exports every
entry point that include/faar.h declares.  No compute call is made here."""
import ctypes as C
import os
import re

import pytest

from paper_2603_22370_b200 import build as faar_build
from paper_2603_22370_b200 import faar

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    faar_build.build()
    return faar.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "faar.h")).read()
    return sorted(set(re.findall(r"FAAR_API\s+[\w\s\*]+?\b(faar_\w+)\s*\(", text)))


def test_header_declares_the_five_named_calls():
    names = declared_symbols()
    for n in ["faar_softquant_init", "faar_softquant_eval", "faar_layer_fwd", "faar_layer_bwd", "faar_round_loss",
              "faar_harden_pack", "faar_layer_step", "faar_layer_ref"]:
        assert n in names


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert len(names) >= 17
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(faar.EXPORTS) == names


def test_status_strings(lib):
    seen = {faar.status_string(i) for i in range(9)}
    assert len(seen) == 9 and "ok" in seen
    assert faar.status_string(99) == "unknown status"


def test_workspace_size_and_shape_validation(lib):
    s = faar.make_shape(128, 256, 1024)
    n = faar.workspace_size(s)
    # header + partials + BF16 W_soft + BF16 dY^T, each region padded
    assert n >= 256 + 128 * 256 * 2 + 128 * 1024 * 2 and n % 1024 == 0
    assert faar.workspace_size(faar.make_shape(128, 256, 1001)) > 0          # ragged T is allowed
    for bad in [faar.make_shape(0, 256, 8), faar.make_shape(8, 250, 8), faar.make_shape(8, 256, 0),
                faar.make_shape(8, -16, 8)]:
        out = C.c_size_t(0)
        assert lib.faar_workspace_size(C.byref(bad), C.byref(out)) == faar.ERR_SHAPE
    assert lib.faar_workspace_size(None, C.byref(C.c_size_t(0))) == faar.ERR_INVALID_ARG
    assert lib.faar_workspace_size(C.byref(s), None) == faar.ERR_INVALID_ARG


def test_null_context_is_rejected_without_touching_a_device(lib):
    s = faar.make_shape(16, 16, 8)
    z = C.c_void_p(0)
    assert lib.faar_softquant_init(z, C.byref(s), z, C.c_float(0), z, z, z, z, z, C.c_size_t(0)) == faar.ERR_INVALID_ARG
    assert lib.faar_layer_step(z, C.byref(s), z, z, z, z, z, z, z, z, z, z, z, z, C.c_size_t(0)) == faar.ERR_INVALID_ARG
    assert lib.faar_harden_pack(z, C.byref(s), z, z, z, z, z, z, z, z, 0) == faar.ERR_INVALID_ARG
    assert lib.faar_create(None, 0, z) == faar.ERR_INVALID_ARG
    assert lib.faar_last_cuda_error(z) == 0


def test_binding_declares_argument_types_for_every_export(lib):
    """Every export has its result and argument types set in the binding, with as many arguments as the
    header's declaration (so no call relies on ctypes' default int promotion)."""
    text = open(os.path.join(ROOT, "include", "faar.h")).read()
    for name in declared_symbols():
        m = re.search(r"FAAR_API\s+[\w\s\*]+?\b" + name + r"\s*\(([^;]*?)\)\s*;", text, re.S)
        assert m, name
        params = m.group(1).strip()
        n_params = 0 if params in ("", "void") else params.count(",") + 1
        fn = getattr(lib, name)
        assert fn.argtypes is not None and len(fn.argtypes) == n_params, (name, n_params, fn.argtypes)
        assert fn.restype is not None


def test_debug_build_exports_the_same_symbols():
    """The bounds-checking build (-DFAAR_DEBUG) is the same library with checked epilogue stores."""
    path = faar_build.build(debug=True)
    dbg = C.CDLL(path)
    for n in declared_symbols():
        assert hasattr(dbg, n), n
