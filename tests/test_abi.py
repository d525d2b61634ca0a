"""CPU-only checks of the boundary: the shared library loads, exports every function that
include/dart.h declares, the header is plain C whose struct layouts match the ctypes
mirrors, and argument validation that needs no GPU answers with error codes."""
import ctypes as C
import os
import re
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "dart.h")


@pytest.fixture(scope="module")
def binding():
    from paper_2601_19278_b200 import build
    build.build()
    from paper_2601_19278_b200 import binding as b
    return b


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dart_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_function(binding):
    lib = binding.lib()
    names = _declared_functions()
    assert {"dart_draft_init", "dart_draft_step", "dart_build_tree", "dart_draft_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in dart.h but not exported"
    assert sorted(binding.EXPORTS) == [n for n in names if n in binding.EXPORTS]
    assert set(binding.EXPORTS) <= set(names)


def test_header_is_plain_c_and_layouts_match_ctypes(binding, tmp_path):
    src = tmp_path / "sz.c"
    src.write_text(
        '#include <stdio.h>\n#include <stddef.h>\n#include "dart.h"\n'
        "int main(void){printf(\"%zu %zu %zu %zu %zu %zu %zu %zu %zu %zu %zu %zu\\n\", sizeof(dart_config), sizeof(dart_weights),"
        " sizeof(dart_ngram_host), sizeof(dart_step_in), sizeof(dart_step_out), sizeof(dart_tree_in), sizeof(dart_tree_out),"
        " offsetof(dart_config, philox_seed), offsetof(dart_step_in, step_counter), offsetof(dart_tree_in, topk_ids),"
        " sizeof(dart_host_io), offsetof(dart_host_io, out_dev));return 0;}\n")
    exe = tmp_path / "sz"
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    got = [int(x) for x in subprocess.check_output([str(exe)]).split()]
    b = binding
    want = [C.sizeof(b.DartConfig), C.sizeof(b.DartWeights), C.sizeof(b.DartNgramHost), C.sizeof(b.DartStepIn),
            C.sizeof(b.DartStepOut), C.sizeof(b.DartTreeIn), C.sizeof(b.DartTreeOut), b.DartConfig.philox_seed.offset,
            b.DartStepIn.step_counter.offset, b.DartTreeIn.topk_ids.offset, C.sizeof(b.DartHostIo), b.DartHostIo.out_dev.offset]
    assert got == want


def test_status_strings_and_workspace_size(binding):
    from paper_2601_19278_b200 import synthetic as syn
    lib = binding.lib()
    assert lib.dart_status_string(0) == b"DART_OK"
    assert lib.dart_status_string(-4) == b"DART_ERR_CAPACITY"
    assert lib.dart_status_string(-99) == b"DART_ERR_UNKNOWN"
    small = binding.workspace_bytes(binding.make_config(syn.WORKLOADS["C1"]))
    big = binding.workspace_bytes(binding.make_config(syn.WORKLOADS["C5"]))
    assert 0 < small < big < 2 << 30
    bad = binding.make_config(syn.WORKLOADS["C1"], head_dim=96)
    assert binding.workspace_bytes(bad) == 0
    bad = binding.make_config(syn.WORKLOADS["C1"], vocab=4100)          # not a multiple of 16
    assert binding.workspace_bytes(bad) == 0
    bad = binding.make_config(syn.WORKLOADS["C1"])
    bad.struct_size = 12
    assert binding.workspace_bytes(bad) == 0


def test_argument_errors_are_reported_without_a_gpu(binding):
    from paper_2601_19278_b200 import synthetic as syn
    lib = binding.lib()
    h = C.c_void_p()
    cfg = binding.make_config(syn.WORKLOADS["C1"])
    assert lib.dart_draft_init(C.byref(cfg), None, None, C.byref(h)) == binding.DART_ERR_INVALID_ARG
    assert not h
    w = binding.DartWeights()                                          # all NULL pointers
    assert lib.dart_draft_init(C.byref(cfg), C.byref(w), None, C.byref(h)) == binding.DART_ERR_INVALID_ARG
    for n in binding.WEIGHT_NAMES:
        setattr(w, n, 0x1010)                                          # 16-byte aligned only: 32 are needed
    assert lib.dart_draft_init(C.byref(cfg), C.byref(w), None, C.byref(h)) == binding.DART_ERR_INVALID_ARG
    assert lib.dart_draft_step(None, None, None, None) == binding.DART_ERR_INVALID_ARG
    assert lib.dart_build_tree(None, None, None, None) == binding.DART_ERR_INVALID_ARG
    assert lib.dart_draft_destroy(None) == binding.DART_OK
    assert lib.dart_step_launch_count(None, 1, 1) == 0


def test_missing_library_fails_loudly(binding, monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libdart.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()


def test_product_code_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2601_19278_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+\.*oracle\b", text, flags=re.M), f"{f} imports the oracle"
                assert not re.search(r"#include\s+[\"<].*oracle", text), f"{f} includes an oracle file"
