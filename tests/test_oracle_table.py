"""Pins for the oracle's brute-force neighborhood table (Eq. s2_neighborhood_attention; App. B.3)."""
import math
import os

import numpy as np
import pytest

from oracle import sna_oracle as orc

EQ, GL = orc.EQUIANGULAR, orc.LEGENDRE_GAUSS
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "tiny_tables.txt")


def _read_golden():
    cases, cur = [], None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "case":
            cur = {"name": tok[1], "rows": {}}
            for kv in tok[2:]:
                key, val = kv.split("=")
                cur[key] = float(val) if key == "theta_cutoff" else int(val)
            cases.append(cur)
        elif tok[0] == "row":
            cur["rows"][int(tok[1])] = [tuple(int(x) for x in t.split(":")) for t in tok[3:]]
    return cases


@pytest.mark.parametrize("case", _read_golden(), ids=lambda c: c["name"])
def test_hand_derived_tiny_tables(case):
    g = orc.geometry(case["nlat_in"], case["nlon_in"], case["nlat_out"], case["nlon_out"],
                     case["grid_in"], case["grid_out"], case["theta_cutoff"])
    for h in range(case["nlat_out"]):
        got = list(zip(g.lat_in[g.row_ptr[h]:g.row_ptr[h + 1]].tolist(),
                       g.lon_off[g.row_ptr[h]:g.row_ptr[h + 1]].tolist()))
        assert got == case["rows"][h], h


def _haversine_table(grid_in, nlat_in, nlon_in, grid_out, nlat_out, theta_c):
    """Independent formulation: haversine distance instead of arccos of a dot product."""
    ti, to = orc.colatitudes(grid_in, nlat_in), orc.colatitudes(grid_out, nlat_out)
    phi = 2 * math.pi * np.arange(nlon_in) / nlon_in
    rows = []
    for h in range(nlat_out):
        lat_o, lat_i = math.pi / 2 - to[h], math.pi / 2 - ti
        a = np.sin((lat_i[:, None] - lat_o) / 2) ** 2 + np.cos(lat_o) * np.cos(lat_i)[:, None] * np.sin(phi[None, :] / 2) ** 2
        d = 2 * np.arcsin(np.sqrt(np.clip(a, 0, 1)))
        hp, wp = np.nonzero(d <= theta_c + 1e-10)
        rows.append(list(zip(hp.tolist(), wp.tolist())))
    return rows


@pytest.mark.parametrize("args", [
    (EQ, 32, 64, EQ, 32, 64, 0.3),
    (EQ, 33, 64, EQ, 17, 32, 2 * math.pi / 16),
    (GL, 24, 48, GL, 24, 48, 0.37),
    (GL, 20, 40, EQ, 11, 20, 0.5),
    (EQ, 64, 128, EQ, 64, 128, 4 * math.pi / 63),      # exact ties on the meridian and at the pole rings
])
def test_second_distance_formula_gives_the_same_table(args):
    gi, nlat_in, nlon_in, go, nlat_out, nlon_out, th = args
    g = orc.geometry(nlat_in, nlon_in, nlat_out, nlon_out, gi, go, th)
    rows = _haversine_table(gi, nlat_in, nlon_in, go, nlat_out, th)
    assert g.nnz == sum(len(r) for r in rows)
    for h in range(nlat_out):
        got = list(zip(g.lat_in[g.row_ptr[h]:g.row_ptr[h + 1]].tolist(), g.lon_off[g.row_ptr[h]:g.row_ptr[h + 1]].tolist()))
        assert got == rows[h]


def test_ties_on_the_boundary_are_members():
    # cutoff = exactly 2 grid spacings: the ring two rows away on the meridian is at distance == cutoff
    nlat, nlon = 17, 32
    g = orc.geometry(nlat, nlon, nlat, nlon, EQ, EQ, 2 * math.pi / (nlat - 1))
    h = 8
    row = set(zip(g.lat_in[g.row_ptr[h]:g.row_ptr[h + 1]].tolist(), g.lon_off[g.row_ptr[h]:g.row_ptr[h + 1]].tolist()))
    assert (h - 2, 0) in row and (h + 2, 0) in row and (h - 3, 0) not in row
    # along the equator d = phi exactly: offsets +-1 are inside (pi/16 < pi/8), +-2 tie (2pi/16 == cutoff)
    assert (h, 2) in row and (h, nlon - 2) in row and (h, 3) not in row


def test_structure_symmetric_windows_and_mirror():
    g = orc.geometry(33, 64, 33, 64, EQ, EQ, 0.41)
    for h in range(33):
        lat = g.lat_in[g.row_ptr[h]:g.row_ptr[h + 1]]
        off = g.lon_off[g.row_ptr[h]:g.row_ptr[h + 1]]
        assert np.all(np.diff(lat) >= 0)
        for hp in np.unique(lat):
            o = set(off[lat == hp].tolist())
            assert 0 in o
            assert o == {(-x) % 64 for x in o}, "window must be symmetric about offset 0"
            m = (len(o) - 1) // 2
            if len(o) < 64:
                assert o == {x % 64 for x in range(-m, m + 1)}, "window must be contiguous"
        # north-south mirror
        hm = 32 - h
        latm = g.lat_in[g.row_ptr[hm]:g.row_ptr[hm + 1]]
        offm = g.lon_off[g.row_ptr[hm]:g.row_ptr[hm + 1]]
        assert sorted(zip((32 - lat).tolist(), off.tolist())) == sorted(zip(latm.tolist(), offm.tolist()))


def test_cutoff_below_grid_spacing_selects_only_the_point_itself():
    nlat, nlon = 9, 16
    g = orc.geometry(nlat, nlon, nlat, nlon, EQ, EQ, 0.05)
    for h in range(nlat):
        row = list(zip(g.lat_in[g.row_ptr[h]:g.row_ptr[h + 1]].tolist(), g.lon_off[g.row_ptr[h]:g.row_ptr[h + 1]].tolist()))
        if h in (0, nlat - 1):          # all points of a pole ring are the same physical point
            assert row == [(h, w) for w in range(nlon)]
        else:
            assert row == [(h, 0)]


def test_cutoff_pi_selects_everything():
    g = orc.geometry(6, 12, 5, 6, EQ, GL, math.pi)
    assert g.nnz == 5 * 6 * 12
    assert np.array_equal(g.lat_in[:72], np.repeat(np.arange(6), 12))
    assert np.array_equal(g.lon_off[:72], np.tile(np.arange(12), 6))


@pytest.mark.parametrize("args", [(EQ, 64, 128, 0.2), (GL, 48, 96, 0.3), (EQ, 128, 256, 4 * math.pi / 127)])
def test_disc_area_band(args):
    # sum of the quadrature weights inside the disc approximates the cap area 2pi(1 - cos theta_c)
    grid, nlat, nlon, th = args
    g = orc.geometry(nlat, nlon, nlat, nlon, grid, grid, th)
    cap = 2 * math.pi * (1 - math.cos(th))
    ratios = np.array([g.omega[g.lat_in[g.row_ptr[h]:g.row_ptr[h + 1]]].sum() / cap for h in range(nlat)])
    assert ratios.min() > 0.6 and ratios.max() < 1.4
    assert abs(np.median(ratios) - 1.0) < 0.1
    gp = orc.geometry(8, 16, 8, 16, grid, grid, math.pi)
    assert abs(gp.omega[gp.lat_in[:gp.row_ptr[1]]].sum() - 4 * math.pi) < 1e-12


def test_table_sizes_of_the_five_benchmark_configurations():
    # independent of the CUDA library: these counts must be reproduced by its planner bit for bit
    assert orc.geometry(32, 64, 32, 64, EQ, EQ, 0.3).nnz == 2334
    assert orc.geometry(128, 256, 128, 256, EQ, EQ, 4 * math.pi / 127).nnz == 22406
    assert orc.geometry(64, 128, 64, 128, EQ, EQ, math.pi).nnz == 524288


def test_errors():
    with pytest.raises(orc.OracleError) as e:
        orc.geometry(8, 16, 8, 5, EQ, EQ, 0.5)          # nlon_in not a multiple of nlon_out
    assert e.value.code == 1
    with pytest.raises(orc.OracleError) as e:
        orc.geometry(5, 8, 16, 8, EQ, GL, 0.02)         # some output rows see no input point
    assert e.value.code == 3
    with pytest.raises(orc.OracleError) as e:
        orc.geometry(17, 32, 17, 32, EQ, EQ, 2 * math.pi / 16 + 1e-10)   # a near-tie inside the ambiguity band
    assert e.value.code == 2
