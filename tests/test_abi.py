"""The C-ABI library loads without a GPU and exports every symbol include/dte.h declares;
host-only entry points behave as documented."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2608_00455_b200 as dte

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "dte.h")).read()
    return sorted(set(re.findall(r"DTE_API[^;(]*?\b(dte_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert len(names) >= 12
    assert sorted(names) == sorted(dte.SYMBOLS)
    L = ctypes.CDLL(dte.library_path()) if os.path.exists(dte.library_path()) else dte.lib()
    for n in names:
        assert hasattr(L, n), n


@pytest.mark.parametrize("args", [(1, 1e-6, 0.9, 0.999, 1e-8, 0.01), (100, 1e-6, 0.9, 0.999, 1e-8, 0.01),
                                  (500, 1e-4, 0.9, 0.999, 1e-8, 0.1), (7, 3e-3, 0.5, 0.5, 0.0, 0.0),
                                  (165, 1e-5, 0.95, 0.98, 1e-6, 0.05)])
def test_constants_bit_identical_to_oracle(args):
    a = dte.dte_derive_constants(*args)
    b = oracle.derive_constants(*args)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


@pytest.mark.parametrize("args", [(0, 1e-6, 0.9, 0.999, 1e-8, 0.01), (1, 1e-6, 1.0, 0.999, 1e-8, 0.01),
                                  (1, 1e-6, 0.9, -0.1, 1e-8, 0.01), (1, 2.0, 0.9, 0.999, 1e-8, 0.5),
                                  (1, 1e-6, 0.9, 0.999, -1e-8, 0.01), (1, float("nan"), 0.9, 0.999, 1e-8, 0.01),
                                  (1, 1e-6, 0.0, 0.999, 1e-8, 0.01 * 0 + float("inf"))])
def test_bad_hyper_parameters_are_rejected(args):
    with pytest.raises(dte.DteError) as e:
        dte.dte_derive_constants(*args)
    assert e.value.status == 1


def test_status_strings():
    L = dte.lib()
    assert L.dte_status_string(0) == b"ok"
    assert L.dte_status_string(2) == b"inconsistent layout"


def test_compute_calls_fail_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        dte.Layout([(4, 4)], [16], [(0, 0, 0, 0, 4, 4, 0, 4, 0, 0)])


@pytest.mark.parametrize("fmt", [0, 1, 2])
@pytest.mark.parametrize("chunk_entries", [8, 64, 4096])
def test_chunk_bounds_cover_what_the_oracle_writes(fmt, chunk_entries):
    # host-only sizing helpers: never smaller than the stream the oracle serialises
    rng = np.random.default_rng(chunk_entries + fmt)
    L = dte.lib()
    for _ in range(20):
        lens = rng.integers(0, 3 * chunk_entries + 2, rng.integers(1, 12))
        lp = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
        n = int(lp[-1])
        stream, d = oracle.pack_chunks(lp, np.arange(n, dtype=np.uint32), np.zeros(n, np.uint16),
                                       chunk_entries, fmt)
        assert d.shape[0] - 1 <= L.dte_chunk_count_bound(lens.size, n, chunk_entries)
        assert stream.size <= L.dte_chunk_bytes_bound(lens.size, n, chunk_entries, fmt)
    assert L.dte_chunk_count_bound(3, 100, 0) == 0


C_PROGRAM = r"""
#include <stdio.h>
#include <string.h>
#include "dte.h"

int main(void) {
    float c[5];
    unsigned int bits[5];
    dte_status s = dte_derive_constants(100, 1e-6, 0.9, 0.999, 1e-8, 0.01, c);
    if (s != DTE_OK) return 2;
    memcpy(bits, c, sizeof bits);
    printf("%08x %08x %08x %08x %08x\n", bits[0], bits[1], bits[2], bits[3], bits[4]);
    s = dte_derive_constants(0, 1e-6, 0.9, 0.999, 1e-8, 0.01, c);          /* step 0: refused */
    printf("%d %s\n", (int)s, dte_status_string(s));
    return dte_layout_num_lists(NULL) == 0 ? 0 : 3;
}
"""


def test_header_is_plain_c_and_the_library_links_from_a_c_program(tmp_path):
    """The boundary is a C ABI: the header compiles as strict C99 (and as C++11), and a C program
    built with gcc alone links against the library and calls its host-only entry points."""
    import shutil
    import subprocess
    if not shutil.which("gcc"):
        pytest.skip("no gcc")
    inc = os.path.join(ROOT, "include")
    hdr = os.path.join(inc, "dte.h")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-x", "c", hdr], check=True)
    subprocess.run(["g++", "-std=c++11", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-x", "c++", hdr], check=True)
    lib = dte.library_path()
    if not os.path.exists(lib):
        dte.lib()
    src = tmp_path / "use_dte.c"
    src.write_text(C_PROGRAM)
    exe = tmp_path / "use_dte"
    libdir = os.path.dirname(lib)
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", inc, str(src), "-o", str(exe),
                    "-L", libdir, "-l:" + os.path.basename(lib), "-Wl,-rpath," + libdir], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split("\n")
    want = oracle.derive_constants(100, 1e-6, 0.9, 0.999, 1e-8, 0.01).view(np.uint32)
    assert out[0].split() == [f"{int(x):08x}" for x in want[:5]]
    assert out[1] == "1 invalid argument"
