"""CPU tests of the C-ABI library: it loads, exports what the header declares, and its host planner
reproduces the oracle's grids, weights and tables bit for bit (no GPU, no compute calls)."""
import ctypes
import math
import os
import re

import numpy as np
import pytest

from oracle import sna_oracle as orc
from paper_2505_11157_b200 import sna
from paper_2505_11157_b200.synthetic import WORKLOADS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
EQ, GL, TZ = 0, 1, 2


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sna.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sna_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_functions()
    assert "sna_plan_create" in names and "sna_forward" in names and "sna_backward" in names and len(names) >= 14
    lib = ctypes.CDLL(sna.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in sna.h but not exported"
    # and the binding names every one of them
    for name in names:
        assert name in sna._SIGNATURES, f"binding lacks {name}"


def test_status_strings():
    assert sna._lib.sna_status_string(0) == b"SNA_OK"
    assert sna._lib.sna_status_string(6) == b"SNA_ERR_AMBIGUOUS_TIE"


CASES = {
    "c1": (32, 64, 32, 64, EQ, EQ, 0.3),
    "c2": (128, 256, 128, 256, EQ, EQ, 4 * math.pi / 127),
    "c5": (64, 128, 64, 128, EQ, EQ, math.pi),
    "down2": (33, 64, 17, 32, EQ, EQ, 2 * math.pi / 16),
    "down4_mixed": (24, 48, 9, 12, GL, EQ, 0.6),
    "gl": (24, 48, 24, 48, GL, GL, 0.37),
    "gl_c4_like": (61, 120, 61, 120, GL, GL, 5 * math.pi / 60),
    "odd_nlon": (10, 15, 10, 15, EQ, EQ, 0.8),
    "tiny": (4, 8, 4, 8, EQ, EQ, 1.1),
    "wide": (16, 32, 16, 32, EQ, EQ, 2.5),
    "trapezoid": (24, 48, 24, 48, TZ, TZ, 0.4),
    "trapezoid_down2_from_gl": (24, 48, 12, 24, GL, TZ, 0.6),
    "trapezoid_global": (8, 16, 8, 16, TZ, TZ, math.pi),
}


@pytest.mark.parametrize("name", list(CASES))
def test_planner_matches_oracle_bit_for_bit(name):
    args = CASES[name]
    g = orc.geometry(*args)
    with sna.Plan(*args, host_only=True) as p:
        assert p.nnz == g.nnz
        row_ptr, lat, off = p.table()
        assert np.array_equal(row_ptr, g.row_ptr)
        assert np.array_equal(lat, g.lat_in)
        assert np.array_equal(off, g.lon_off)
        ti, to = p.colatitudes()
        assert np.allclose(ti, orc.colatitudes(args[4], args[0]), rtol=0, atol=2e-15)
        assert np.allclose(to, orc.colatitudes(args[5], args[2]), rtol=0, atol=2e-15)
        assert np.allclose(p.quad_weights(), g.omega, rtol=1e-13, atol=0)
        if args[4] != TZ:
            assert abs(p.quad_weights().sum() * args[1] - 4 * math.pi) < 1e-12
        else:
            assert p.quad_weights()[0] == 0.0
        # transposed table, rebuilt here from the oracle's table
        ps = args[1] // args[3]
        t_ptr, t_lat, t_off = p.table_transposed()
        h_of_entry = np.repeat(np.arange(args[2]), np.diff(g.row_ptr))
        expect = []
        for hin in range(args[0]):
            for r in range(ps):
                sel = (g.lat_in == hin) & (g.lon_off % ps == r)
                expect.append(sorted(zip(h_of_entry[sel].tolist(), g.lon_off[sel].tolist())))
        assert t_ptr[-1] == g.nnz
        for row, exp in enumerate(expect):
            got = list(zip(t_lat[t_ptr[row]:t_ptr[row + 1]].tolist(), t_off[t_ptr[row]:t_ptr[row + 1]].tolist()))
            assert got == exp, row


def test_planner_matches_oracle_on_random_problems():
    """Sixty seeded random problems (all three grids, ps in 1..4, arbitrary latitude counts and cutoffs): the planner's
    table, or its refusal, must be the oracle's."""
    rng = np.random.default_rng(2505)
    status_of = {2: sna.SNA_ERR_AMBIGUOUS_TIE, 3: sna.SNA_ERR_EMPTY_NEIGHBORHOOD}
    compared = refused = 0
    for _ in range(60):
        ps = int(rng.integers(1, 5))
        nlon_out = int(rng.integers(3, 40))
        nlat_in, nlat_out = int(rng.integers(2, 40)), int(rng.integers(2, 40))
        gi, go = int(rng.integers(0, 3)), int(rng.integers(0, 3))
        theta = float(rng.uniform(0.02, 1.0)) if rng.random() < 0.8 else float(rng.uniform(1.0, 3.3))
        args = (nlat_in, nlon_out * ps, nlat_out, nlon_out, gi, go, theta)
        try:
            g = orc.geometry(*args)
        except orc.OracleError as e:
            with pytest.raises(sna.SnaError) as pe:
                sna.Plan(*args, host_only=True)
            assert pe.value.status == status_of[e.code], args
            refused += 1
            continue
        with sna.Plan(*args, host_only=True) as p:
            row_ptr, lat, off = p.table()
            assert np.array_equal(row_ptr, g.row_ptr) and np.array_equal(lat, g.lat_in) and np.array_equal(off, g.lon_off), args
            assert np.allclose(p.quad_weights(), g.omega, rtol=1e-13, atol=0), args
        compared += 1
    assert compared >= 30 and refused >= 1


def test_headline_table_sizes():
    for name, nnz in (("c3", 53800), ("c4", 98995)):
        wl = WORKLOADS[name]
        with sna.Plan(wl.nlat_in, wl.nlon_in, wl.nlat_out, wl.nlon_out, wl.grid_in, wl.grid_out, wl.theta_cutoff,
                      host_only=True) as p:
            assert p.nnz == nnz


@pytest.mark.parametrize("args, status", [
    ((8, 16, 8, 5, EQ, EQ, 0.5), sna.SNA_ERR_UNSUPPORTED),
    ((8, 16, 8, 16, EQ, 5, 0.5), sna.SNA_ERR_UNSUPPORTED),
    ((1, 16, 8, 16, EQ, EQ, 0.5), sna.SNA_ERR_INVALID_ARG),
    ((8, 16, 8, 16, EQ, EQ, 0.0), sna.SNA_ERR_INVALID_ARG),
    ((8, 16, 8, 16, EQ, EQ, float("nan")), sna.SNA_ERR_INVALID_ARG),
    ((5, 8, 16, 8, EQ, GL, 0.02), sna.SNA_ERR_EMPTY_NEIGHBORHOOD),
    ((16, 32, 16, 32, TZ, TZ, 0.05), sna.SNA_ERR_EMPTY_NEIGHBORHOOD),   # the pole's disc holds only the zero-weight pole ring
    ((17, 32, 17, 32, EQ, EQ, 2 * math.pi / 16 + 1e-10), sna.SNA_ERR_AMBIGUOUS_TIE),
])
def test_plan_errors(args, status):
    with pytest.raises(sna.SnaError) as e:
        sna.Plan(*args, host_only=True)
    assert e.value.status == status
    assert str(e.value)


def test_host_only_plan_refuses_to_compute():
    with sna.Plan(8, 16, 8, 16, EQ, EQ, 0.5, host_only=True) as p:
        assert sna._lib.sna_forward(p.handle, 16, 16, 16, 16, 1, 1, 4, None) == sna.SNA_ERR_INVALID_ARG
        assert sna._lib.sna_forward(None, 16, 16, 16, 16, 1, 1, 4, None) == sna.SNA_ERR_INVALID_ARG
        assert sna.sna_workspace_bytes(p.handle, 2, 3, 4) == 2 * 3 * 8 * 16 * 2 * 4
        assert sna.sna_workspace_bytes(p.handle, 0, 3, 4) == 0


def test_binding_refuses_wrong_dtype_shape_and_device_before_any_launch():
    """The kernels trust raw pointers, so the binding must stop malformed tensors on the host.  Nothing is
    launched here: the plan is host-only and every call fails validation first."""
    import torch
    with sna.Plan(8, 16, 8, 16, EQ, EQ, 0.9, host_only=True) as p:
        q = torch.zeros(1, 2, 8, 16, 8)
        k = torch.zeros(1, 2, 8, 16, 8)
        with pytest.raises(ValueError, match="float32"):
            p.forward(q, k, k.half())
        with pytest.raises(ValueError, match="float32"):
            p.backward(q, k, k, q.double())
        with pytest.raises(ValueError, match="shape"):
            p.forward(q, k, torch.zeros(1, 2, 8, 15, 8))
        with pytest.raises(ValueError, match="shape"):
            p.backward(q, k, k, q, lse=torch.zeros(1, 2, 8, 15))
        with pytest.raises(ValueError, match="shape"):
            p.backward(q, k, k, q, dk=torch.zeros(1, 2, 8, 16, 4))
        with pytest.raises(ValueError, match="do not match the plan"):
            p.forward(torch.zeros(1, 2, 8, 15, 8), k, k)
        with pytest.raises(ValueError, match="CUDA"):
            p.forward(q, k, k)          # right dtype and shape, but host memory


def test_unsupported_channel_counts_are_refused_on_the_host():
    with sna.Plan(8, 16, 8, 16, EQ, EQ, 0.9, host_only=True) as p:
        for C in (0, 3, 6, 130, 132):
            st = sna._lib.sna_forward(p.handle, 16, 16, 16, 16, 1, 1, C, None)
            assert st in (sna.SNA_ERR_INVALID_ARG, sna.SNA_ERR_UNSUPPORTED), C
