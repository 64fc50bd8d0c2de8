"""The C-ABI library loads without a GPU and exports every entry point that
include/jackpot.h declares (no compute call is made here)."""
import ctypes
import os
import re
import subprocess

from paper_2602_06107_b200 import binding as B
from paper_2602_06107_b200 import build as jp_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "jackpot.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(jp_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_header_declares_the_calls_the_binding_uses():
    decl = declared_functions()
    assert "jp_obrs_forward" in decl and "jp_obrs_backward" in decl
    assert set(B.EXPORTS) <= set(decl), set(B.EXPORTS) - set(decl)


def test_library_exports_every_declared_symbol():
    path = jp_build.build()
    lib = ctypes.CDLL(path)
    missing = [n for n in declared_functions() if not hasattr(lib, n)]
    assert not missing, missing


def test_status_strings_and_sizes_without_a_device():
    lib = B.load()
    assert lib.jp_status_string(0) == b"ok"
    assert b"argument" in lib.jp_status_string(-1)
    # workspace sizing is host arithmetic: grows with rows and with k
    a = lib.jp_obrs_workspace_bytes(1024, 151936, 32)
    b = lib.jp_obrs_workspace_bytes(2048, 151936, 32)
    c = lib.jp_obrs_workspace_bytes(1024, 151936, 64)
    assert 0 < a < b and a < c
    assert lib.jp_obrs_workspace_bytes(-1, 10, 1) == 0


def test_ctypes_structs_match_the_header(tmp_path):
    """sizeof / offsetof as gcc sees the header against the ctypes mirrors."""
    src = tmp_path / "sz.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "jackpot.h"\n'
                   'int main(void){printf("%zu %zu %zu %zu %zu %zu %zu\\n", sizeof(jp_stats), sizeof(jp_obrs_desc),'
                   ' sizeof(jp_obrs_bwd_desc), offsetof(jp_obrs_desc, token_offset), offsetof(jp_obrs_desc, lse_policy),'
                   ' offsetof(jp_stats, status), offsetof(jp_obrs_bwd_desc, record_offset));return 0;}\n')
    exe = tmp_path / "sz"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    got = [int(x) for x in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()]
    want = [ctypes.sizeof(B.jp_stats), ctypes.sizeof(B.jp_obrs_desc), ctypes.sizeof(B.jp_obrs_bwd_desc),
            B.jp_obrs_desc.token_offset.offset, B.jp_obrs_desc.lse_policy.offset, B.jp_stats.status.offset,
            B.jp_obrs_bwd_desc.record_offset.offset]
    assert got == want
