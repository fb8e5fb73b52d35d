"""The C-ABI shared library: it loads without a GPU, exports every symbol the
header declares, and its structs have the sizes the Python binding assumes."""
import ctypes
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "baoc.h")


@pytest.fixture(scope="module")
def binding():
    from paper_2605_04711_b200 import build
    build.build()
    from paper_2605_04711_b200 import binding as B
    return B


def _declared():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(baoc_[a-z_0-9]+)\s*\(", src)))


def test_every_declared_symbol_is_exported(binding):
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = _declared()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_struct_sizes_match_the_header(binding, tmp_path):
    prog = tmp_path / "sizes.c"
    prog.write_text('#include <stdio.h>\n#include "baoc.h"\nint main(void){printf("%zu %zu %zu %zu %zu\\n",'
                    'sizeof(baoc_block_t),sizeof(baoc_config_t),sizeof(baoc_opts_t),sizeof(baoc_block_stats_t),'
                    'sizeof(baoc_info_t));return 0;}\n')
    exe = tmp_path / "sizes"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), str(prog), "-o", str(exe)], check=True)
    got = [int(x) for x in subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()]
    B = binding
    want = [ctypes.sizeof(B.Block), ctypes.sizeof(B.Config), ctypes.sizeof(B.Opts), ctypes.sizeof(B.BlockStats),
            ctypes.sizeof(B.Info)]
    assert got == want


def test_header_is_plain_c(tmp_path):
    prog = tmp_path / "c89.c"
    prog.write_text('#include "baoc.h"\nint main(void){return 0;}\n')
    subprocess.run(["gcc", "-std=c99", "-pedantic", "-Werror", "-I", os.path.join(ROOT, "include"), "-c", str(prog),
                    "-o", str(tmp_path / "c89.o")], check=True)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2605_04711_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".cpp", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"(import|from|include)\s+\S*oracle", text), f
    # and the oracle does not import the product
    text = open(os.path.join(ROOT, "oracle", "baoc_oracle.py")).read()
    assert "paper_2605_04711_b200" not in text and "ctypes" not in text
