"""CPU-side checks of the C-ABI library: it builds, loads and exports every symbol the header
declares; the ctypes mirrors of the structs match the C layout; host-side argument checks work
without a GPU."""
import ctypes as C
import os
import re
import subprocess
import sys
import tempfile

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "pact.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2504_08966_b200 import build
    build.build()
    from paper_2504_08966_b200 import binding
    return binding.lib()


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pact_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2504_08966_b200 import binding
    names = _declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(binding.EXPORTS)


def test_struct_layouts_match_the_header():
    from paper_2504_08966_b200 import binding
    src = r'''
#include <stdio.h>
#include <stddef.h>
#include "pact.h"
int main(void) {
  printf("%zu %zu %zu %zu %zu %zu %zu\n", sizeof(pact_params), offsetof(pact_params, d_c), offsetof(pact_params, flags),
         sizeof(pact_image), offsetof(pact_image, P), offsetof(pact_image, H_out), offsetof(pact_image, counters));
  return 0;
}'''
    with tempfile.TemporaryDirectory() as td:
        cfile, exe = os.path.join(td, "t.c"), os.path.join(td, "t")
        open(cfile, "w").write(src)
        subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), cfile, "-o", exe])
        got = [int(x) for x in subprocess.check_output([exe]).split()]
    P, I = binding.Params, binding.ImageDesc
    want = [C.sizeof(P), P.d_c.offset, P.flags.offset, C.sizeof(I), I.P.offset, I.H_out.offset, I.counters.offset]
    assert got == want


def test_host_side_checks_without_a_gpu(lib):
    import torch
    assert lib.pact_workspace_bytes(None, 1, 10) == 0
    assert lib.pact_host_staging_bytes(None, 10, 10) == 0
    assert lib.pact_status_string(0) == b"ok" and b"workspace" in lib.pact_status_string(-3)
    h = C.c_void_p()
    assert lib.pact_create(C.byref(h), 128, 4, 3, 16, 0, 0) == -1          # heads do not divide
    assert lib.pact_create(C.byref(h), 128, 4, 4, 12, 0, 0) == -2          # d_h not a multiple of 8 for bf16
    assert lib.pact_create(None, 128, 4, 4, 16, 0, 0) == -1
    if not torch.cuda.is_available():
        st = lib.pact_create(C.byref(h), 128, 4, 4, 16, 0, 0)
        assert st == -4 and not h.value                                     # no device: a clean CUDA error
    assert lib.pact_reduce(None, None, 0, None, 0, None, 0, None) == -1


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2504_08966_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle", text, flags=re.M), f
                assert "pact_oracle" not in text and "oracle/" not in text, f
