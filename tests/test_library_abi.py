"""The C-ABI library builds, loads and exports every symbol the header declares; host-side
argument checks answer without a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2606_01927_b200 import _build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "albireo_sample.h")


@pytest.fixture(scope="module")
def lib():
    return C.CDLL(_build.build())


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(albireo_[a-z_]+)\s*\(", text)))


def test_header_declares_the_three_calls_and_helpers():
    names = declared_functions()
    for need in ("albireo_sample_init", "albireo_sample", "albireo_sample_destroy"):
        assert need in names


def test_every_declared_symbol_is_exported(lib):
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_exports():
    from paper_2606_01927_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()


def test_workspace_size_is_a_pure_function(lib):
    f = lib.albireo_sample_workspace_bytes
    f.restype = C.c_size_t
    f.argtypes = [C.c_int32, C.c_int32, C.c_int64]
    a = f(256, 152064, 0)
    b = f(256, 152064, 1 << 20)
    assert a > 0 and a % 256 == 0 and b >= a + 4 * (1 << 20) and b % 256 == 0
    assert f(-1, 10, 0) == 0
    g = lib.albireo_sample_host_staging_bytes
    g.restype = C.c_size_t
    g.argtypes = [C.c_int32, C.c_int32, C.c_int64]
    assert g(256, 152064, 0) >= 256 * 152064 * 4


def test_init_rejects_bad_arguments_before_touching_cuda(lib):
    init = lib.albireo_sample_init
    init.restype = C.c_int
    init.argtypes = [C.POINTER(C.c_void_p), C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_void_p, C.c_size_t]
    h = C.c_void_p(123)
    assert init(C.byref(h), 0, 0, 100, 0, None, 0) == -1 and not h.value          # max_rows < 1
    assert init(C.byref(h), 0, 8, 100, 0, None, 0) == -1                          # NULL workspace
    assert init(C.byref(h), 0, 8, 1 << 22, 0, C.c_void_p(256), 1 << 20) == -4     # vocabulary too large
    assert init(C.byref(h), 0, 8, 100, 0, C.c_void_p(257), 1 << 20) == -1         # misaligned workspace
    assert init(None, 0, 8, 100, 0, C.c_void_p(256), 1 << 20) == -1
    lib.albireo_sample_destroy.argtypes = [C.c_void_p]
    assert lib.albireo_sample_destroy(None) == 0
    lib.albireo_last_error.restype = C.c_char_p
    lib.albireo_last_error.argtypes = [C.c_void_p]
    assert lib.albireo_last_error(None) == b""


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2606_01927_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h", ".cpp")):
                src = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in src.lower() or fn == "workloads.py", fn


def test_binding_struct_and_constants_match_the_header(tmp_path):
    """The ctypes mirror of albireo_sample_ext_t has the C layout (size and every field offset), and the
    binding's constants are the header's: checked by compiling the header with the host C compiler."""
    import subprocess
    from paper_2606_01927_b200 import binding
    fields = [f[0] for f in binding.SampleExt._fields_]
    prog = ['#include <stdio.h>', '#include <stddef.h>', '#include "albireo_sample.h"', 'int main(void) {',
            '  printf("sizeof %zu\\n", sizeof(albireo_sample_ext_t));']
    prog += [f'  printf("{f} %zu\\n", offsetof(albireo_sample_ext_t, {f}));' for f in fields]
    for name in ("ALBIREO_F32", "ALBIREO_BF16", "ALBIREO_F16", "ALBIREO_MAX_VOCAB", "ALBIREO_MAX_NUM_TOP",
                 "ALBIREO_FLAG_FORCE_GENERAL", "ALBIREO_FLAG_TOPK_KEEP_TIES", "ALBIREO_FLAG_LOGPROB_FULL_VOCAB",
                 "ALBIREO_FLAG_PROGRAMMATIC_LAUNCH", "ALBIREO_FIXED_MAX_HISTORY", "ALBIREO_OK"):
        prog.append(f'  printf("{name} %lld\\n", (long long){name});')
    prog += ['  return 0;', '}']
    src = tmp_path / "layout.c"
    src.write_text("\n".join(prog))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = dict(line.split() for line in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines())
    assert int(out["sizeof"]) == C.sizeof(binding.SampleExt)
    for f in fields:
        assert int(out[f]) == getattr(binding.SampleExt, f).offset, f
    assert (int(out["ALBIREO_F32"]), int(out["ALBIREO_BF16"]), int(out["ALBIREO_F16"])) == (binding.F32, binding.BF16, binding.F16)
    assert int(out["ALBIREO_MAX_VOCAB"]) == binding.MAX_VOCAB and int(out["ALBIREO_MAX_NUM_TOP"]) == binding.MAX_NUM_TOP
    assert int(out["ALBIREO_FLAG_FORCE_GENERAL"]) == binding.FLAG_FORCE_GENERAL
    assert int(out["ALBIREO_FLAG_TOPK_KEEP_TIES"]) == binding.FLAG_TOPK_KEEP_TIES
    assert int(out["ALBIREO_FLAG_LOGPROB_FULL_VOCAB"]) == binding.FLAG_LOGPROB_FULL_VOCAB
    assert int(out["ALBIREO_FLAG_PROGRAMMATIC_LAUNCH"]) == binding.FLAG_PROGRAMMATIC_LAUNCH
    assert int(out["ALBIREO_FIXED_MAX_HISTORY"]) == binding.FIXED_MAX_HISTORY and int(out["ALBIREO_OK"]) == binding.OK
