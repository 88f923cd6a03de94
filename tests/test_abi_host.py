"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and the integer planner matches the oracle bit for bit."""
import ctypes
import itertools
import os
import re

import numpy as np
import pytest

from oracle import reference as orc
from paper_2609_04774_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def test_library_exports_every_declared_symbol(lib):
    from paper_2609_04774_b200 import cache_manager
    for hname, exports in (("cpattn.h", binding.EXPORTS), ("cpcache.h", cache_manager.EXPORTS)):
        header = open(os.path.join(ROOT, "include", hname)).read()
        header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
        declared = set(re.findall(r"\b(cp_[a-z_0-9]+)\s*\(", header))
        assert declared, "no declarations found in " + hname
        assert declared == set(exports), hname
        for name in declared:
            assert hasattr(lib, name), name


def test_struct_layouts_match_header():
    assert ctypes.sizeof(binding.cp_shard_plan) == 56
    assert ctypes.sizeof(binding.cp_kv_cache) == 64


def test_cp_plan_bit_exact_against_oracle(lib):
    cases = list(itertools.product(list(range(1, 70)) + [127, 128, 129, 1000, 4096], [0, 1, 64, 12288], [1, 2, 3, 4, 5, 8]))
    cases += [(1024, 0, 2), (4096, 12288, 4), (131072, 0, 8), (32768, 32768, 8), (65536, 64, 7)]
    for R, P, C in cases:
        assert binding.cp_plan(R, P, C) == orc.plan(R, P, C), (R, P, C)


def test_cp_plan_rejects_bad_arguments(lib):
    for args in [(0, 0, 1), (-3, 0, 2), (5, -1, 1), (5, 0, 0)]:
        with pytest.raises(binding.CpError) as e:
            binding.cp_plan(*args)
        assert e.value.code == binding.CP_ERR_INVALID_ARG
    assert b"cp_plan" in lib.cp_last_error()
    assert lib.cp_strerror(-5) == b"CP_ERR_TIMEOUT"


def test_workspace_bytes(lib):
    small = binding.cp_workspace_bytes([1024], [2], 8)
    big = binding.cp_workspace_bytes([131072], [8], 32)
    assert 50e6 < small < 60e6                       # dominated by the fixed partial-result space
    # 32 bytes per query tile + 16 bytes per (tile, head) unit (one head per unit in the worst case)
    assert big - small == pytest.approx((1040 - 12) * 32 + (1040 * 32 - 12 * 8) * 16, abs=1024)
    assert small % 256 == 0 and big % 256 == 0
    assert binding.cp_workspace_bytes([0], [1], 8) == 0
    assert binding.cp_workspace_bytes([64], [1], 0) == 0


def test_gpu_calls_fail_cleanly_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(binding.CpError) as e:
        binding.Context(0)
    assert e.value.code in (binding.CP_ERR_CUDA, binding.CP_ERR_INVALID_ARG)


def test_headers_compile_as_c99_and_link_from_c(lib, tmp_path):
    # the boundary is a C ABI: both public headers must be valid C (not only C++), and a plain C program linked
    # against the library must get the planner's numbers (compared with the oracle's plan)
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no gcc on this machine")
    src = tmp_path / "use_cpattn.c"
    src.write_text(
        '#include "cpattn.h"\n#include "cpcache.h"\n#include <stdio.h>\n'
        "int main(void) {\n"
        "    cp_shard_plan plan[4];\n"
        "    int rc = cp_plan(4096, 12288, 4, plan);\n"
        "    for (int k = 0; k < 4 && rc == 0; ++k)\n"
        '        printf("%lld %lld %lld %lld %lld %lld %llu\\n", (long long)plan[k].q_begin[0], (long long)plan[k].q_end[0],\n'
        "               (long long)plan[k].q_begin[1], (long long)plan[k].q_end[1], (long long)plan[k].kv_end[0],\n"
        "               (long long)plan[k].kv_end[1], (unsigned long long)plan[k].pairs);\n"
        '    printf("%s\\n", cp_strerror(rc));\n'
        "    return rc;\n}\n")
    exe = tmp_path / "use_cpattn"
    libdir = os.path.dirname(build.LIB_PATH)
    subprocess.check_call([gcc, "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(build.ROOT, "include"),
                           str(src), "-o", str(exe), "-L", libdir, "-l:" + os.path.basename(build.LIB_PATH),
                           "-Wl,-rpath," + libdir])
    out = subprocess.check_output([str(exe)], text=True).split("\n")
    ref = orc.plan(4096, 12288, 4)
    for k in range(4):
        got = [int(x) for x in out[k].split()]
        assert got == [ref[k]["q_begin"][0], ref[k]["q_end"][0], ref[k]["q_begin"][1], ref[k]["q_end"][1],
                       ref[k]["kv_end"][0], ref[k]["kv_end"][1], ref[k]["pairs"]]
    assert out[4] == "CP_OK"
