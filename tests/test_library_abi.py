"""The C-ABI library builds, loads and exports every symbol include/hoccl.h and include/hoccl_diag.h declare (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import diag as hd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions(header="hoccl.h"):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hoccl_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    L = hb.lib()
    names = _declared_functions()
    assert len(names) >= 25
    for n in names:
        assert hasattr(L, n), n
    assert sorted(hb.EXPORTS) == names, (set(names) ^ set(hb.EXPORTS))
    # the diagnostics header and its binding
    hd.lib()
    dnames = _declared_functions("hoccl_diag.h")
    assert len(dnames) >= 15 and not set(dnames) & set(names)
    for n in dnames:
        assert hasattr(L, n), n
    assert sorted(hd.EXPORTS) == dnames, (set(dnames) ^ set(hd.EXPORTS))


def test_error_strings_and_sizes():
    assert hb.error_string(hb.OK) == "ok"
    for code in range(1, 9):
        assert hb.error_string(code) and hb.error_string(code) != "ok"
    assert hb.scratch_bytes(1, 1000, "fp32") == 0
    assert hb.scratch_bytes(8, 0, "bf16") == 0
    # 2 slots per rank, each one ring chunk + slack, padded to 256
    n = 13_107_200
    b = hb.scratch_bytes(8, n, "bf16")
    chunk = n // 8 * 2
    assert b >= 2 * 8 * chunk and b <= 2 * 8 * (chunk + chunk // 64 + 512)
    assert b % 256 == 0


def test_argument_errors_need_no_device():
    L = hb.lib()
    h = ctypes.c_void_p()
    assert L.hoccl_comm_init(None, 4, 0) == hb.ERR_INVALID_ARG
    assert L.hoccl_comm_init(ctypes.byref(h), 0, 0) == hb.ERR_INVALID_ARG
    assert L.hoccl_comm_init(ctypes.byref(h), 65, 0) == hb.ERR_INVALID_ARG
    assert L.hoccl_comm_destroy(None) == hb.ERR_INVALID_ARG
    assert hd.lib().hoccl_sum_launch(None, None, None, 4, 0, 8, None) == hb.ERR_INVALID_ARG
    assert hd.lib().hoccl_sum_launch(16, 32, 48, 4, 7, 8, None) == hb.ERR_UNSUPPORTED
    assert hd.lib().hoccl_sum_launch(18, 32, 48, 4, 0, 8, None) == hb.ERR_INVALID_ARG      # misaligned for fp32
    p = ctypes.c_void_p()
    assert hd.lib().hoccl_plan_build(ctypes.byref(p), 0, 0, 10, 0, 0, 4096, 8, None) == hb.ERR_INVALID_ARG
    assert hd.lib().hoccl_plan_build(ctypes.byref(p), 0, 4, 10, 9, 0, 4096, 8, None) == hb.ERR_UNSUPPORTED


def test_no_device_fails_loudly():
    """Without a CUDA device the product path reports an error; it never falls back to the CPU."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(hb.HocclError) as ei:
        hb.Comm(4, 0)
    assert ei.value.code == hb.ERR_CUDA


def test_header_is_plain_c_and_a_c_program_links_against_the_library(tmp_path):
    """The boundary is a C ABI: the header compiles as strict C99 (and as C++), and a C program that names every entry
    point links against libhoccl.so and runs its host-only calls (no device needed)."""
    import shutil
    import subprocess
    if not shutil.which("gcc"):
        pytest.skip("no C compiler")
    inc = os.path.join(ROOT, "include")
    libdir = os.path.dirname(hb.library_path())
    names = _declared_functions() + _declared_functions("hoccl_diag.h")
    src = tmp_path / "use_hoccl.c"
    refs = "\n".join("  fns[n++] = (void (*)(void))%s;" % n for n in names)
    src.write_text('#include <stdio.h>\n#include <string.h>\n#include "hoccl.h"\n#include "hoccl_diag.h"\nint main(void) {\n  void (*fns[128])(void);\n  int n = 0;\n'
                   + refs + '\n  if (strcmp(hoccl_error_string(HOCCL_OK), "ok") != 0) return 2;\n'
                   '  if (hoccl_scratch_bytes(1, 1000, HOCCL_FLOAT32) != 0) return 3;\n'
                   '  if (hoccl_comm_set_path(0, HOCCL_PATH_CE) != HOCCL_ERR_INVALID_ARG) return 4;\n'
                   '  for (int k = 0; k < n; k++) if (!fns[k]) return 5;\n'
                   '  printf("%d entry points\\n", n);\n  return 0;\n}\n')
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-fsyntax-only", "-I", inc, str(src)], check=True)
    subprocess.run(["g++", "-std=c++11", "-Wall", "-Werror", "-fsyntax-only", "-x", "c++", "-I", inc, str(src)], check=True)
    exe = tmp_path / "use_hoccl"
    subprocess.run(["gcc", "-std=c99", "-I", inc, str(src), "-o", str(exe), "-L", libdir, "-lhoccl", "-Wl,-rpath," + libdir], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout
    assert out.strip() == "%d entry points" % len(names)
