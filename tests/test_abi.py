"""The C-ABI boundary without a GPU: the library loads, exports every declared symbol, and its host
logic (permutation generator, workspace planning, argument checks) behaves as the header states."""
import ctypes
import math
import os
import re

import numpy as np
import pytest

from oracle import mhclite_oracle as O
from paper_2601_05732_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"MHCLITE_API\s+[\w\s\*]+?\b(mhc\w+)\s*\(", src)
    return names


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    names = _declared()
    assert len(names) >= 19 and len(set(names)) == len(names)
    for name in names:
        assert hasattr(lib, name), name
    # the Python binding marshals exactly the declared entry points
    assert set(binding.SIGNATURES) == set(names)


def test_declared_argument_counts_match_binding():
    src = open(os.path.join(ROOT, "include", "mhclite.h")).read()
    for name, (_, args) in binding.SIGNATURES.items():
        m = re.search(r"\b" + name + r"\s*\(([^;]*?)\)\s*;", src, flags=re.S)
        assert m, name
        declared = [a for a in m.group(1).split(",") if a.strip() and a.strip() != "void"]
        assert len(declared) == len(args), name


@pytest.mark.parametrize("n", [2, 3, 4, 5])
def test_perm_table_bit_exact(n):
    got = binding.perm_table(n)
    ref = O.perm_table(n)
    assert got.dtype == np.uint8 and got.shape == ref.shape
    assert (got == ref).all()


def test_perm_table_rejects_bad_n():
    lib = binding.load()
    buf = (ctypes.c_uint8 * 1024)()
    assert lib.mhclite_perm_table(1, buf) == binding.ERR_BAD_ARG
    assert lib.mhclite_perm_table(6, buf) == binding.ERR_BAD_ARG
    assert lib.mhclite_perm_table(4, None) == binding.ERR_BAD_ARG


def test_workspace_bytes():
    wb = binding.workspace_bytes
    assert wb(4, 1024, 0) >= 0 and wb(4, 1024, 16384) > wb(4, 1024, 1024) > 0
    assert wb(4, 1024, 16384) % 256 == 0
    assert wb(1, 1024, 10) == 0 and wb(6, 1024, 10) == 0 and wb(4, 1024, -1) == 0   # rejected -> 0
    assert wb(4, 1024, 16384) < 64 << 20
    ws = binding.load().mhclite_workspace_bytes_subset
    assert 0 < ws(5, 1536, 4096, 8) < ws(5, 1536, 4096, 64) <= wb(5, 1536, 4096)      # fewer columns, less scratch
    assert ws(5, 1536, 4096, 0) == 0 and ws(5, 1536, 4096, 121) == 0 and ws(4, 64, 10, 25) == 0


def test_status_strings_and_null_context():
    lib = binding.load()
    assert binding.status_string(0) == "ok"
    for code in (-1, -2, -3, -4):
        assert binding.status_string(code) not in ("ok", "unknown status")
    assert lib.mhclite_destroy(None) == binding.ERR_BAD_ARG
    assert lib.mhclite_premix_fwd(None, 4, None, None, None, None) == binding.ERR_BAD_ARG
    h = ctypes.c_void_p()
    assert lib.mhclite_create(ctypes.byref(h), 7, 1024, 0) == binding.ERR_BAD_ARG     # n out of range
    assert lib.mhclite_create(ctypes.byref(h), 4, 1023, 0) == binding.ERR_BAD_ARG     # C % 8 != 0
    assert lib.mhclite_create(None, 4, 1024, 0) == binding.ERR_BAD_ARG


def test_no_cpu_fallback_without_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        binding.MhcLite(4, 64)
    h = ctypes.c_void_p()
    assert binding.load().mhclite_create(ctypes.byref(h), 4, 64, 0) == binding.ERR_CUDA
