"""The C-ABI library loads and exports every symbol include/fp4attn.h declares (no GPU work)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_04105_b200 import build
    return ctypes.CDLL(build.build())


def _declared():
    text = open(os.path.join(ROOT, "include", "fp4attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fp4attn_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert "fp4attn_quantize" in names and "fp4attn_fwd" in names
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_symbols():
    from paper_2609_04105_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_size_queries_and_status_strings(lib):
    lib.fp4attn_packed_bytes.restype = ctypes.c_size_t
    lib.fp4attn_scale_bytes.restype = ctypes.c_size_t
    lib.fp4attn_quantize_workspace_bytes.restype = ctypes.c_size_t
    lib.fp4attn_status_string.restype = ctypes.c_char_p
    assert lib.fp4attn_packed_bytes(4, 16, 4096, 128) == 4 * 16 * 4096 * 128 // 2
    # Q/K MXFP4 d=128: 4 scale bytes per row -> one 512-byte atom per 128 rows
    assert lib.fp4attn_scale_bytes(0, 0, 1, 2, 256, 128) == 2 * 2 * 512
    # NVFP4 d=128: 8 scale columns -> two atoms per 128 rows;  d=64: one
    assert lib.fp4attn_scale_bytes(1, 1, 1, 1, 128, 128) == 1024
    assert lib.fp4attn_scale_bytes(1, 1, 1, 1, 128, 64) == 512
    # V: rows d (padded to 128), columns N/32 -> one atom per 128 keys
    assert lib.fp4attn_scale_bytes(0, 2, 1, 1, 1024, 64) == 8 * 512
    assert lib.fp4attn_scale_bytes(1, 2, 1, 1, 1024, 64) == 0          # V is never NVFP4
    assert lib.fp4attn_scale_bytes(0, 0, 1, 1, 100, 128) == 0          # N not a multiple of 128
    assert lib.fp4attn_quantize_workspace_bytes(0, 0, 1, 1, 128, 128) == 0
    assert lib.fp4attn_quantize_workspace_bytes(1, 0, 1, 1, 128, 128) > 0
    assert lib.fp4attn_status_string(0) == b"ok"
    assert b"unknown" in lib.fp4attn_status_string(99)


def test_host_detectable_errors_return_codes_without_a_gpu(lib):
    lib.fp4attn_quantize.restype = ctypes.c_int
    vp = ctypes.c_void_p
    args = lambda x, fmt, role, N, d, G=None: (vp(x), fmt, role, 1, 1, N, d, vp(0x1000), vp(0x2000), G, None,
                                               ctypes.c_size_t(0), None)
    assert lib.fp4attn_quantize(*args(0, 0, 0, 128, 128)) == 1            # NULL input
    assert lib.fp4attn_quantize(*args(0x1000, 5, 0, 128, 128)) == 1       # unknown format
    assert lib.fp4attn_quantize(*args(0x1000, 0, 0, 100, 128)) == 2       # unsupported N
    assert lib.fp4attn_quantize(*args(0x1000, 0, 0, 128, 96)) == 2        # unsupported d
    assert lib.fp4attn_quantize(*args(0x1004, 0, 0, 128, 128)) == 4       # misaligned
    assert lib.fp4attn_quantize(*args(0x1000, 1, 2, 128, 128, vp(0x3000))) == 1   # NVFP4 V
    assert lib.fp4attn_quantize(*args(0x1000, 1, 0, 128, 128, vp(0x3000))) == 5   # NVFP4 without workspace
    lib.fp4attn_softmax_arith_probe.restype = ctypes.c_int
    assert lib.fp4attn_softmax_arith_probe(0, 0, 0, vp(0x1000), None) == 1          # no iterations
    assert lib.fp4attn_softmax_arith_probe(0, 0, 1 << 21, vp(0x1000), None) == 1    # more than the cap
    assert lib.fp4attn_softmax_arith_probe(2, 0x0101, 16, vp(0x1000), None) == 1    # a pattern no kernel has
    assert lib.fp4attn_softmax_arith_probe(0, 0, 16, None, None) == 1               # nowhere to write


def test_header_is_plain_c_and_the_struct_layout_matches_the_binding(lib, tmp_path):
    """The boundary is usable from C: the header compiles as strict C99, a C program links against the
    library and calls it, and the operand struct it sees has the layout the Python binding marshals."""
    import shutil
    import subprocess
    from paper_2609_04105_b200 import binding, build
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    fields = [n for n, _ in binding._Operands._fields_]
    src = tmp_path / "abi.c"
    lines = ['#include <stddef.h>', '#include <stdio.h>', '#include <string.h>', '#include "fp4attn.h"', 'int main(void) {',
             '  fp4attn_operands ops;', '  memset(&ops, 0, sizeof ops);',
             '  printf("sizeof %zu\\n", sizeof(fp4attn_operands));']
    lines += [f'  printf("{n} %zu\\n", offsetof(fp4attn_operands, {n}));' for n in fields]
    lines += ['  printf("version %d\\n", fp4attn_version());',
              '  printf("packed %zu\\n", fp4attn_packed_bytes(4, 16, 4096, 128));',
              '  printf("null_ops %d\\n", fp4attn_fwd(NULL, 1, 1, 128, 128, NULL, NULL, NULL, NULL));',
              '  printf("status %s\\n", fp4attn_status_string(FP4ATTN_ERR_INVALID_ARG));',
              '  return 0;', '}']
    src.write_text("\n".join(lines) + "\n")
    libpath = build.build()
    exe = tmp_path / "abi"
    subprocess.run([gcc, "-std=c99", "-pedantic", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src),
                    "-o", str(exe), libpath, f"-Wl,-rpath,{os.path.dirname(libpath)}"], check=True)
    out = dict(l.split(" ", 1) for l in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines())
    assert int(out["sizeof"]) == ctypes.sizeof(binding._Operands)
    for n in fields:
        assert int(out[n]) == getattr(binding._Operands, n).offset, n
    assert int(out["version"]) == lib.fp4attn_version()
    assert int(out["packed"]) == 4 * 16 * 4096 * 128 // 2
    assert int(out["null_ops"]) == binding.ERR_INVALID_ARG
    assert out["status"] == "invalid argument"
