"""The C-ABI library builds, loads and exports every symbol the header declares (CPU only;
no compute call is made without a GPU)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for h in sorted(os.listdir(inc)):
        if not h.endswith(".h"):
            continue
        text = open(os.path.join(inc, h)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(kb_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_public_header_keeps_hooks_out():
    text = open(os.path.join(ROOT, "include", "kb.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    for hook in ("kb_ctx_set_grid", "kb_ctx_set_small_path", "kb_ctx_set_wins_algo", "kb_alu_probe",
                 "kb_ctx_enable_timing", "kb_ctx_fail_next_allocs", "kb_ctx_selftest_wait"):
        assert hook not in text


def test_header_declares_the_three_calls():
    names = declared_functions()
    for must in ("kb_screen", "kb_adjudicate", "kb_select", "kb_ctx_create", "kb_ctx_destroy"):
        assert must in names


def test_library_exports_every_declared_symbol():
    from paper_2608_02611_b200 import build, binding
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in include/ but not exported"
    assert sorted(binding.EXPORTS) == declared_functions()
    binding.load()


def test_result_record_layout_matches_header():
    from paper_2608_02611_b200 import binding
    assert binding.RESULT_DTYPE.itemsize == 48
    assert [binding.RESULT_DTYPE.fields[n][1] for n in binding.RESULT_DTYPE.names] == \
        [0, 8, 16, 24, 32, 36, 40, 44]


def test_no_device_is_a_clean_error():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    from paper_2608_02611_b200 import binding
    with pytest.raises(binding.KbError):
        binding.Context(0)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2608_02611_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text, f
                assert "kb_oracle" not in text, f


def test_header_is_plain_c99_and_a_c_program_links(tmp_path):
    """include/kb.h compiles as C99 (no C++ or CUDA types in the boundary) with the record
    sizes it documents, and a C translation unit that calls an entry point links against the
    library.  The program is not run: without a GPU kb_ctx_create would only report that."""
    import subprocess
    from paper_2608_02611_b200 import build
    lib_path = build.build()
    src = tmp_path / "use_kb.c"
    src.write_text(
        '#include "kb_hooks.h"\n'
        "typedef char rec32[sizeof(kb_screen_result) == 48 ? 1 : -1];\n"
        "typedef char rec64[sizeof(kb_screen_result_f64) == 56 ? 1 : -1];\n"
        "int main(void) {\n"
        "  kb_ctx* ctx = 0;\n"
        "  kb_status st = kb_ctx_create(0, &ctx);\n"
        "  if (st == KB_OK) kb_ctx_destroy(ctx);\n"
        "  return (int)st;\n"
        "}\n")
    exe = tmp_path / "use_kb"
    cmd = ["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
           str(src), lib_path, "-o", str(exe), "-Wl,-rpath," + os.path.dirname(lib_path),
           "-Wl,--allow-shlib-undefined"]
    done = subprocess.run(cmd, capture_output=True, text=True)
    assert done.returncode == 0, done.stderr
