"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_2108_02191_b200 as robe
from oracle import robe_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "robe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(robe_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 11
    lib = C.CDLL(robe.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(robe.EXPORTS) == names
    for n in names:
        assert callable(getattr(robe, n)), f"binding lacks {n}"


def test_binding_has_no_fallback_import():
    src = open(os.path.join(ROOT, "paper_2108_02191_b200", "binding.py")).read()
    assert "oracle" not in src
    for f in os.listdir(os.path.join(ROOT, "paper_2108_02191_b200", "csrc")):
        assert "oracle" not in open(os.path.join(ROOT, "paper_2108_02191_b200", "csrc", f)).read()


@pytest.mark.parametrize("args", [
    (0, 1, 1, 1), (10, 0, 4, 1), (10, 4, 0, 1), (10, 4, 4, 0), (10, 6, 4, 1), (10, 12, 4, 1), (3, 2, 4, 1),
    (2**32, 4, 16, 1), (2**32 - 15, 4, 16, 1), (10**6, 4, 40000, 1),
])
def test_create_rejects_bad_shapes(args):
    with pytest.raises(robe.RobeError) as ei:
        robe.robe_create(*args, 1)
    assert ei.value.status == robe.ROBE_ERR_INVALID_ARG


def test_create_accepts_limits_and_constants_match_oracle():
    for M, Z, d, T in [(1, 1, 1, 1), (2**32 - 16, 4, 16, 26), (4096, 4, 16, 4), (100, 100, 100, 3)]:
        for seed in (0, 0x0B0F, 2**64 - 1):
            h = robe.robe_create(M, Z, d, T, seed)
            k = robe.robe_get_hash_constants(h)
            assert k == [int(v) for v in orc.hash_constants(seed)]
            robe.robe_destroy(h)


def test_options_and_errors_without_device():
    h = robe.robe_create(4096, 4, 16, 4, 7)
    for key, val in [(robe.ROBE_OPT_SIGN, 2), (robe.ROBE_OPT_BWD_MODE, 5), (99, 0),
                     (robe.ROBE_OPT_VALIDATE, -1), (robe.ROBE_OPT_FWD_KERNEL, 5), (robe.ROBE_OPT_BWD_KERNEL, 7),
                     (robe.ROBE_OPT_INDEX_TYPE, 2), (robe.ROBE_OPT_BAG_LAYOUT, 2)]:
        with pytest.raises(robe.RobeError):
            robe.robe_set_option(h, key, val)
    robe.robe_set_option(h, robe.ROBE_OPT_SIGN, 1)
    robe.robe_set_option(h, robe.ROBE_OPT_SIGN, 0)
    robe.robe_set_option(h, robe.ROBE_OPT_INDEX_TYPE, robe.ROBE_I32)
    robe.robe_set_option(h, robe.ROBE_OPT_INDEX_TYPE, robe.ROBE_I64)
    robe.robe_set_option(h, robe.ROBE_OPT_BAG_LAYOUT, robe.ROBE_BAGS_TABLE_MAJOR)
    robe.robe_set_option(h, robe.ROBE_OPT_BAG_LAYOUT, robe.ROBE_BAGS_SAMPLE_MAJOR)
    lib = robe.binding.raw()
    # forward before attach: no array (dummy non-null pointers are never dereferenced)
    dummy = C.c_void_p(0x1000)
    assert lib.robe_forward(h, dummy, None, 2, 8, dummy, None) == robe.ROBE_ERR_NO_ARRAY
    # null pointers and inconsistent sizes
    assert lib.robe_forward(h, None, None, 2, 8, dummy, None) == robe.ROBE_ERR_INVALID_ARG
    assert lib.robe_forward(h, dummy, None, 2, 7, dummy, None) == robe.ROBE_ERR_INVALID_ARG
    assert lib.robe_forward(h, dummy, None, -1, 8, dummy, None) == robe.ROBE_ERR_INVALID_ARG
    assert lib.robe_forward(None, dummy, None, 2, 8, dummy, None) == robe.ROBE_ERR_INVALID_ARG
    assert lib.robe_backward(h, None, dummy, None, 2, 8, dummy, 0.0, None, 0, None) == robe.ROBE_ERR_INVALID_ARG
    # fused SGD needs the array
    assert lib.robe_backward(h, dummy, dummy, None, 2, 8, None, 0.1, None, 0, None) == robe.ROBE_ERR_NO_ARRAY
    # misaligned array pointer
    assert lib.robe_attach_array(h, C.c_void_p(0x1004), robe.ROBE_F32) == robe.ROBE_ERR_INVALID_ARG
    assert lib.robe_attach_array(h, dummy, 7) == robe.ROBE_ERR_INVALID_ARG
    # deterministic mode: workspace is required and sized by the library
    robe.robe_set_option(h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_DETERMINISTIC)
    need = robe.robe_backward_workspace_bytes(h, 2, 8)
    assert need >= 4 * 4 * 8 * 4 and need % 256 == 0
    assert lib.robe_backward(h, dummy, dummy, None, 2, 8, dummy, 0.0, None, 0, None) == robe.ROBE_ERR_WORKSPACE
    assert lib.robe_backward(h, dummy, dummy, None, 2, 8, dummy, 0.0, dummy, need // 2, None) == robe.ROBE_ERR_WORKSPACE
    robe.robe_set_option(h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_ATOMIC)
    assert robe.robe_backward_workspace_bytes(h, 2, 8) == 0
    assert robe.robe_status_string(robe.ROBE_ERR_WORKSPACE).startswith("workspace")
    assert robe.robe_status_string(0) == "ok"
    robe.robe_destroy(h)


def test_workspace_grows_with_blocks():
    h = robe.robe_create(25_000_000, 1, 128, 26, 1)
    robe.robe_set_option(h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_DETERMINISTIC)
    a = robe.robe_backward_workspace_bytes(h, 1024, 1024 * 26)
    b = robe.robe_backward_workspace_bytes(h, 2048, 2048 * 26)
    assert b > a >= 16 * 1024 * 26 * 128
    robe.robe_destroy(h)


def test_sort_based_variants_refuse_sizes_beyond_their_32_bit_numbering():
    # block numbers, bag numbers and gradient positions are 32-bit in the binned / deterministic /
    # Adam paths: larger calls are refused before anything is launched (dummy pointers are never read)
    lib = robe.binding.raw()
    dummy = C.c_void_p(0x1000)
    h = robe.robe_create(1 << 20, 4, 16, 1, 3)        # C = 4 blocks per id
    assert lib.robe_attach_array(h, dummy, robe.ROBE_F32) == robe.ROBE_OK
    big = 1 << 30                                     # 2^30 ids -> 2^32 blocks
    for mode in (robe.ROBE_BWD_DETERMINISTIC, robe.ROBE_BWD_BINNED):
        robe.robe_set_option(h, robe.ROBE_OPT_BWD_MODE, mode)
        assert lib.robe_backward(h, dummy, dummy, None, big, big, dummy, 0.0, dummy, 1 << 40, None) \
            == robe.ROBE_ERR_UNSUPPORTED
    assert lib.robe_backward_adam(h, dummy, dummy, None, big, big, dummy, dummy, 0.1, 0.9, 0.999, 1e-8, 1,
                                  dummy, 1 << 40, None) == robe.ROBE_ERR_UNSUPPORTED
    assert lib.robe_backward_deterministic_static(h, dummy, dummy, None, big, big, dummy, 0.0, None) \
        == robe.ROBE_ERR_UNSUPPORTED
    # atomic mode has no such limit on the host side, but still wants consistent sizes
    robe.robe_set_option(h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_ATOMIC)
    assert lib.robe_backward(h, dummy, dummy, None, big, big - 1, dummy, 0.0, None, 0, None) \
        == robe.ROBE_ERR_INVALID_ARG
    robe.robe_destroy(h)


def test_header_is_plain_c_and_cpp(tmp_path):
    # the boundary is a C ABI: the header must compile as C11 and as C++ with nothing but itself
    import subprocess
    inc = os.path.join(ROOT, "include")
    for comp, std, ext in (("gcc", "-std=c11", "c"), ("g++", "-std=c++11", "cpp")):
        src = tmp_path / f"use_robe.{ext}"
        src.write_text('#include "robe.h"\nint main(void) { robe_handle_t h = 0; return robe_destroy(h) == ROBE_OK; }\n')
        r = subprocess.run([comp, std, "-Wall", "-Wextra", "-Werror", "-pedantic", "-fsyntax-only", "-I", inc, str(src)],
                           capture_output=True, text=True)
        assert r.returncode == 0, r.stderr


C_PROGRAM = r"""
#include <stdio.h>
#include <string.h>
#include "robe.h"
int main(void) {
    robe_handle_t h = 0;
    uint64_t k[9];
    if (robe_create(&h, 4096, 4, 16, 4, 7) != ROBE_OK) return 1;
    if (robe_get_hash_constants(h, k) != ROBE_OK || k[0] != ((1ull << 61) - 1)) return 2;
    if (robe_set_option(h, ROBE_OPT_SIGN, 1) != ROBE_OK) return 3;
    if (robe_forward(h, (const void*)0x1000, 0, 2, 8, (float*)0x1000, 0) != ROBE_ERR_NO_ARRAY) return 4;
    if (robe_create(&h, 10, 12, 4, 1, 7) != ROBE_ERR_INVALID_ARG) return 5;  /* Z > d, not a multiple */
    if (strcmp(robe_status_string(ROBE_ERR_WORKSPACE), "workspace missing, misaligned or too small") != 0) return 6;
    printf("%llu\n", (unsigned long long)k[1]);
    return 0;
}
"""


def test_c_program_links_and_calls_the_library(tmp_path):
    # a C caller, not ctypes: compile against include/robe.h, link librobe.so, run the host-only calls
    import subprocess
    src = tmp_path / "caller.c"
    src.write_text(C_PROGRAM)
    exe = tmp_path / "caller"
    lib_dir = os.path.dirname(robe.LIB_PATH)
    r = subprocess.run(["gcc", "-std=c11", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o",
                        str(exe), "-L", lib_dir, "-l:" + os.path.basename(robe.LIB_PATH), "-Wl,-rpath," + lib_dir],
                       capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    r = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert r.returncode == 0, (r.returncode, r.stderr)
    assert int(r.stdout.strip()) == int(orc.hash_constants(7)[1])  # A_h as the oracle draws it
