"""The C-ABI library loads without a GPU, exports everything include/a2cid2.h declares, and its
host-only entry points (graph quantities, parameter prescription, validation) behave."""
import ctypes as C
import math
import os
import re

import numpy as np
import pytest

from oracle import spectral
from paper_2306_08289_b200 import binding as B
from paper_2306_08289_b200 import build as build_mod
from paper_2306_08289_b200 import workload as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def _declared():
    src = open(os.path.join(ROOT, "include", "a2cid2.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(a2cid2_[a-z_0-9]+)\s*\(", src)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared()
    assert len(names) >= 25 and "a2cid2_apply_events" in names and "a2cid2_consensus_distance" in names
    raw = C.CDLL(B.LIB_PATH)
    for nm in names:
        assert hasattr(raw, nm), nm
    assert set(names) == set(B.SIGNATURES), set(names) ^ set(B.SIGNATURES)
    assert B.lib().a2cid2_version().startswith(b"a2cid2")


def test_enumerators_of_the_header_are_those_of_the_binding():
    src = open(os.path.join(ROOT, "include", "a2cid2.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    found = {k: int(v.rstrip("u")) for k, v in re.findall(r"\b(A2_[A-Z0-9_]+)\s*=\s*(-?\d+u?)", src)}
    assert len(found) >= 30
    for name, value in found.items():
        assert getattr(B, name) == value, name


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4", "cfg5"])
def test_graph_quantities_agree_with_checker(name):
    c = W.CONFIGS[name]
    c1, c2 = B.graph_chi(c.n, c.edges(), c.rates())
    eta, alpha, at, o1, o2 = spectral.prescribe(c.n, c.edges(), c.rates())
    assert abs(c1 - o1) < 1e-10 * o1 and abs(c2 - o2) < 1e-10 * o2
    e2, a2, at2 = B.prescribe(c1, c2)
    assert abs(e2 - eta) < 1e-10 * eta and a2 == alpha and abs(at2 - at) < 1e-10 * at
    assert B.prescribe(c1, c2, accelerated=False) == (0.0, 0.5, 0.5)


def test_graph_quantities_irregular_graph_and_errors():
    # a path with unequal rates: not regular, checks the general code path
    edges = np.array([[0, 1], [1, 2], [2, 3], [1, 3]], dtype=np.int32)
    lam = np.array([0.5, 2.0, 1.0, 0.25])
    c1, c2 = B.graph_chi(4, edges, lam)
    L = spectral.laplacian(4, edges, lam)
    assert abs(c1 - spectral.chi1(L)) < 1e-12 and abs(c2 - spectral.chi2(L, edges)) < 1e-12
    with pytest.raises(B.A2Error) as e:
        B.graph_chi(4, np.array([[0, 1], [2, 3]], dtype=np.int32), np.ones(2))  # disconnected
    assert e.value.code == B.A2_EINVAL
    with pytest.raises(B.A2Error) as e:
        B.graph_chi(4, np.array([[0, 4]], dtype=np.int32), np.ones(1))
    assert e.value.code == B.A2_ERANGE
    with pytest.raises(B.A2Error):
        B.graph_chi(4, edges, -lam)


def test_create_validates_without_a_device():
    L = B.lib()
    h = C.c_void_p()
    assert L.a2cid2_create(1, 10, 0.1, 0.5, 0.5, 0.1, B.A2_F32, C.byref(h)) == B.A2_EINVAL
    assert L.a2cid2_create(4, 0, 0.1, 0.5, 0.5, 0.1, B.A2_F32, C.byref(h)) == B.A2_EINVAL
    assert L.a2cid2_create(4, 10, -0.1, 0.5, 0.5, 0.1, B.A2_F32, C.byref(h)) == B.A2_EINVAL
    assert L.a2cid2_create(4, 10, math.nan, 0.5, 0.5, 0.1, B.A2_F32, C.byref(h)) == B.A2_EINVAL
    assert L.a2cid2_create(4, 10, 0.1, 0.5, 0.5, 0.1, 7, C.byref(h)) == B.A2_EINVAL
    assert b"storage" in L.a2cid2_last_error(None)
    assert L.a2cid2_create(4, 10, 0.1, 0.5, 0.5, 0.1, B.A2_BF16, C.byref(h)) == B.A2_OK and h.value
    # nothing is bound: every device call refuses instead of touching memory
    out = C.c_double()
    assert L.a2cid2_consensus_distance(h, math.nan, C.byref(out)) == B.A2_ESTATE
    t = np.zeros(1)
    i = np.zeros(1, dtype=np.int32)
    assert L.a2cid2_apply_events(h, 0, None, None, None, None, 0, None) == B.A2_ESTATE
    assert b"bind" in L.a2cid2_last_error(h)
    tt = np.array([1.0, 2.0, 3.0, 4.0])
    assert L.a2cid2_set_times(h, tt.ctypes.data_as(C.POINTER(C.c_double))) == B.A2_OK
    back = np.zeros(4)
    assert L.a2cid2_times(h, back.ctypes.data_as(C.POINTER(C.c_double))) == B.A2_OK and np.array_equal(back, tt)
    assert L.a2cid2_sync(h) == B.A2_OK
    for v in (B.A2_MSG_BEFORE_MIX, B.A2_NO_MOMENTUM, B.A2_MSG_AFTER_MIX):
        assert L.a2cid2_set_variant(h, v) == B.A2_OK
    assert L.a2cid2_set_variant(h, 3) == B.A2_EINVAL and L.a2cid2_set_variant(h, -1) == B.A2_EINVAL
    for m in (B.A2_LAUNCH_PER_BATCH, B.A2_LAUNCH_COLUMN_SLICES, B.A2_LAUNCH_AUTO):
        assert L.a2cid2_set_launch_mode(h, m) == B.A2_OK
    assert L.a2cid2_set_launch_mode(h, 3) == B.A2_EINVAL and b"launch mode" in L.a2cid2_last_error(h)
    # this handle stores bf16 rows: rounding x once per store instead of once per event is an fp32 matter
    assert L.a2cid2_set_rounding(h, B.A2_ROUND_PER_EVENT) == B.A2_OK
    assert L.a2cid2_set_rounding(h, B.A2_ROUND_PER_STORE) == B.A2_EINVAL and b"fp32" in L.a2cid2_last_error(h)
    assert L.a2cid2_set_rounding(h, 2) == B.A2_EINVAL
    f = C.c_void_p()
    assert L.a2cid2_create(4, 10, 0.1, 0.5, 0.5, 0.1, B.A2_F32, C.byref(f)) == B.A2_OK
    assert L.a2cid2_set_rounding(f, B.A2_ROUND_PER_STORE) == B.A2_OK
    L.a2cid2_destroy(f)
    # binding without an x~ buffer is refused unless the variant has no momentum (checked before any device call)
    dummy = C.c_void_p(4096)
    assert L.a2cid2_bind(h, dummy, None, None, 0, 16, None) == B.A2_EINVAL
    assert b"x_tilde" in L.a2cid2_last_error(h)
    L.a2cid2_destroy(h)
    L.a2cid2_destroy(None)


def test_header_is_plain_c_and_a_c_program_links_against_the_library(tmp_path):
    """The boundary is a C ABI: the header compiles as strict C99 and a C program that only uses
    host-side entry points (no device needed) links against the shared library and runs."""
    import subprocess

    inc = os.path.join(ROOT, "include")
    subprocess.run(["gcc", "-fsyntax-only", "-x", "c", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror",
                    os.path.join(inc, "a2cid2.h")], check=True)
    src = tmp_path / "use_abi.c"
    src.write_text(r"""
#include <stdio.h>
#include "a2cid2.h"
int main(void) {
    int32_t ei[4] = {0, 1, 2, 0}, ej[4] = {1, 2, 3, 3};
    double lam[4] = {1.0, 1.0, 1.0, 1.0}, c1, c2, eta, alpha, at;
    if (a2cid2_graph_chi(4, 4, ei, ej, lam, &c1, &c2) != A2_OK) return 1;
    if (a2cid2_prescribe(c1, c2, 1, &eta, &alpha, &at) != A2_OK) return 2;
    double times[3] = {0.5, 1.0, 1.5};
    int32_t wi[3] = {0, 2, 1}, wj[3] = {1, 3, 2}, slot[3] = {-1, -1, -1};
    a2cid2_sched_t* s = 0;
    if (a2cid2_sched_create(4, 0, 0, 3, times, wi, wj, slot, A2_SCHED_CHAIN, 0, 0, &s) != A2_OK) return 3;
    long long nb = (long long)a2cid2_sched_num_batches(s);
    a2cid2_sched_destroy(s);
    wi[0] = 7;  /* out of range: rejected with a message */
    if (a2cid2_sched_create(4, 0, 0, 3, times, wi, wj, slot, 0, 0, 0, &s) != A2_ERANGE) return 4;
    printf("%.6f %.6f %.6f %.6f %lld %s|%s\n", c1, c2, eta, at, nb, a2cid2_last_error(0), a2cid2_version());
    return 0;
}
""")
    exe = tmp_path / "use_abi"
    libdir = os.path.dirname(B.LIB_PATH)
    subprocess.run(["gcc", "-std=c99", "-I", inc, str(src), "-o", str(exe), "-L", libdir, "-la2cid2",
                    f"-Wl,-rpath,{libdir}"], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()
    c1, c2, eta, at = (float(v) for v in out[:4])
    # ring of 4 with unit rates: chi_1 = 1/2, chi_2 = 3/8
    assert abs(c1 - 0.5) < 1e-6 and abs(c2 - 0.375) < 1e-6 and abs(eta - 1 / (2 * math.sqrt(c1 * c2))) < 1e-5
    assert int(out[4]) == 2 and "out of range" in " ".join(out[5:])
