"""GPU parity: the CUDA path (through the C ABI) against the fp64 CPU oracle on the same seeded inputs.

Gate (stated by the benchmark definition): neighborhood tables bit-exact; normalised max error
max|x - o| / max|o| per tensor <= 1e-5 for the forward output and <= 1e-4 for each of dq, dk, dv.
"""
import math

import numpy as np
import pytest
import torch

from oracle import sna_oracle as orc
from paper_2505_11157_b200 import sna
from paper_2505_11157_b200.synthetic import WORKLOADS, make_inputs, sample_points, small_workload

pytestmark = pytest.mark.gpu

EQ, GL, TZ = 0, 1, 2
FWD_TOL, BWD_TOL = 1e-5, 1e-4


def nerr(x, ref):
    """Normalised max error of a tensor against the oracle's."""
    x = np.asarray(x, dtype=np.float64)
    return float(np.max(np.abs(x - ref)) / np.max(np.abs(ref)))


def perr(x, ref):
    """A finer measure beside the per-tensor gate: per grid point, the 2-norm of the error over the channels divided
    by the 2-norm of the oracle's vector at that point (floored at 1e-3 of the largest such norm), maximum over points.
    One large element elsewhere in the tensor cannot hide an error here."""
    x = np.asarray(x, dtype=np.float64).reshape(ref.shape)
    d = np.linalg.norm(x - ref, axis=-1)
    n = np.linalg.norm(ref, axis=-1)
    return float(np.max(d / np.maximum(n, 1e-3 * n.max())))


PT_FWD_TOL, PT_BWD_TOL = 2e-5, 3e-4      # measured: out <= 6.5e-6; dq <= 1.3e-4 (2 million points of c4), dk <= 5.9e-5, dv <= 2.1e-5


def _geometry(wl):
    return orc.geometry(wl.nlat_in, wl.nlon_in, wl.nlat_out, wl.nlon_out, wl.grid_in, wl.grid_out, wl.theta_cutoff)


def _plan(wl):
    return sna.Plan(wl.nlat_in, wl.nlon_in, wl.nlat_out, wl.nlon_out, wl.grid_in, wl.grid_out, wl.theta_cutoff)


def _dev(*arrays):
    return [torch.from_numpy(a).cuda() for a in arrays]


def _run_gpu(plan, q, k, v, dout, reuse_forward_state=True):
    qd, kd, vd, dd = _dev(q, k, v, dout)
    out, lse = plan.forward(qd, kd, vd, return_lse=True)
    if reuse_forward_state:
        dq, dk, dv = plan.backward(qd, kd, vd, dd, out=out, lse=lse)
    else:
        dq, dk, dv = plan.backward(qd, kd, vd, dd)
    torch.cuda.synchronize()
    sna.sna_plan_check(plan.handle)      # no kernel gave up on a bounded wait
    return [t.cpu().numpy() for t in (out, lse, dq, dk, dv)]


SMALL = [
    # name, nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, theta, B, H, C, seed
    small_workload("eq_c32", 24, 48, 24, 48, EQ, EQ, 0.45, 1, 3, 32, 10),
    small_workload("eq_c32_ragged", 19, 90, 19, 90, EQ, EQ, 0.3, 2, 1, 32, 11),           # 90 is not a tile multiple
    small_workload("eq_down2_c32", 33, 64, 17, 32, EQ, EQ, 2 * math.pi / 16, 1, 2, 32, 12),
    small_workload("gl_c32", 20, 40, 20, 40, GL, GL, 0.5, 2, 2, 32, 13),
    small_workload("gl_to_eq_down4_c16", 24, 48, 9, 12, GL, EQ, 0.6, 1, 2, 16, 14),
    small_workload("eq_c4", 12, 24, 12, 24, EQ, EQ, 0.6, 1, 2, 4, 15),
    small_workload("eq_c8_oddlon", 10, 15, 10, 15, EQ, EQ, 0.8, 1, 1, 8, 16),
    small_workload("eq_c64", 16, 32, 16, 32, EQ, EQ, 0.5, 1, 1, 64, 17),
    small_workload("eq_c128", 12, 24, 12, 24, EQ, EQ, 0.7, 1, 1, 128, 18),
    small_workload("global_c32", 12, 24, 12, 24, EQ, EQ, math.pi, 1, 2, 32, 19),
    small_workload("eq_wide_c32", 40, 160, 40, 160, EQ, EQ, 0.5, 1, 1, 32, 20),           # several tiles per ring
    small_workload("eq_single_neighbor", 9, 16, 9, 16, EQ, EQ, 0.05, 1, 1, 32, 21),       # degenerate: disc = the point itself
    small_workload("eq_down2_wide_c32", 41, 320, 21, 160, EQ, EQ, 0.25, 1, 1, 32, 22),
    small_workload("eq_down3_c32", 25, 96, 13, 32, EQ, EQ, 0.4, 1, 2, 32, 23),             # ps = 3: transposed stream by residue
    small_workload("gl_down4_c32", 24, 160, 12, 40, GL, GL, 0.45, 1, 1, 32, 24),           # ps = 4, nlon_out not a tile multiple
    small_workload("eq_oddlat_c16", 21, 64, 21, 64, EQ, EQ, 0.35, 1, 2, 16, 25),           # odd ring count: last ring group is half empty
    small_workload("eq_c64_wide", 14, 48, 14, 48, EQ, EQ, 0.9, 1, 1, 64, 26),
    small_workload("gl_latratio_2p4_c32", 24, 64, 10, 32, GL, GL, 0.5, 1, 2, 32, 27),      # latitude grids do not nest
    small_workload("eq_to_gl_up_lat_c32", 9, 40, 20, 40, EQ, GL, 0.6, 1, 1, 32, 28),       # more output than input rings
    small_workload("eq_nearly_global_c32", 12, 32, 12, 32, EQ, EQ, 2.6, 1, 1, 32, 29),     # windows wider than half a ring
    small_workload("eq_many_heads_c16", 10, 32, 10, 32, EQ, EQ, 0.5, 3, 7, 16, 30),        # 21 independent slices
    # whole-ring windows everywhere: both dense tensor-core kernels do all the work
    small_workload("global_c32_dense", 14, 64, 14, 64, EQ, EQ, math.pi, 1, 2, 32, 33),
    small_workload("global_ragged_dense", 10, 80, 10, 80, GL, GL, math.pi, 2, 1, 32, 34),  # 80 columns: partial last block; 80 rows < 128
    small_workload("global_down2_dense", 12, 288, 7, 144, EQ, EQ, math.pi, 1, 1, 32, 35),  # 144 rows: two row blocks, the second ragged
    small_workload("polar_heavy_c32", 16, 64, 16, 64, EQ, EQ, 1.2, 1, 2, 32, 36),          # dense and banded windows mixed in every row
    # channel counts that are multiples of 4 but not powers of two (lane groups padded with zero lanes)
    small_workload("eq_c12", 12, 24, 12, 24, EQ, EQ, 0.6, 1, 2, 12, 37),
    small_workload("gl_down2_c24", 17, 64, 9, 32, GL, GL, 0.5, 2, 1, 24, 38),
    small_workload("eq_c48", 10, 40, 10, 40, EQ, EQ, 0.7, 1, 1, 48, 39),
    # the grid as the paper prints it: pole ring of quadrature weight zero (inside discs, contributes nothing, dk = dv = 0)
    small_workload("trapezoid_c32", 24, 48, 24, 48, TZ, TZ, 0.45, 1, 2, 32, 43),
    small_workload("trapezoid_down2_c32", 32, 128, 16, 64, TZ, TZ, 0.5, 1, 2, 32, 44),
    small_workload("trapezoid_polar_heavy_c32", 16, 64, 16, 64, TZ, TZ, 1.2, 1, 2, 32, 45),   # dense and banded windows mixed
    small_workload("trapezoid_c16", 12, 32, 12, 32, TZ, TZ, 0.6, 1, 2, 16, 46),
    small_workload("trapezoid_c12_generic", 12, 24, 12, 24, TZ, GL, 0.6, 1, 2, 12, 47),
    small_workload("trapezoid_global_c32", 12, 64, 12, 64, TZ, TZ, math.pi, 1, 2, 32, 48),
    # windows of 128 columns and more that are not whole rings: masked blocks on the dense kernels, pieces across the seam
    small_workload("wide_windows_c32", 24, 320, 24, 320, EQ, EQ, 0.55, 1, 1, 32, 49),
    small_workload("wide_windows_down2_c32", 33, 384, 17, 192, EQ, EQ, 0.5, 1, 2, 32, 50),
    small_workload("wide_windows_down4_gl_c32", 20, 640, 10, 160, GL, GL, 0.6, 1, 1, 32, 51),
    small_workload("wide_windows_trapezoid_c32", 20, 300, 20, 300, TZ, TZ, 0.6, 2, 1, 32, 52),   # 300: ragged tiles and blocks
]


@pytest.mark.parametrize("wl", SMALL + [WORKLOADS["c1"]], ids=lambda w: w.name)
@pytest.mark.parametrize("reuse", [True, False], ids=["reuse_lse_out", "recompute_stats"])
def test_small_cases_full_comparison(wl, reuse):
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)
    with _plan(wl) as plan:
        row_ptr, lat, off = plan.table()
        assert np.array_equal(row_ptr, g.row_ptr) and np.array_equal(lat, g.lat_in) and np.array_equal(off, g.lon_off)
        out, lse, dq, dk, dv = _run_gpu(plan, q, k, v, dout, reuse)
    N = wl.N
    ref_out, ref_lse = orc.forward(g, q, k, v, return_lse=True)
    rdq, rdk, rdv = orc.backward(g, q, k, v, dout)
    assert nerr(out.reshape(ref_out.shape), ref_out) <= FWD_TOL
    assert np.max(np.abs(lse.reshape(ref_lse.shape) - ref_lse)) <= 1e-5 * max(1.0, np.max(np.abs(ref_lse)))
    assert nerr(dq.reshape(rdq.shape), rdq) <= BWD_TOL
    assert nerr(dk.reshape(rdk.shape), rdk) <= BWD_TOL
    assert nerr(dv.reshape(rdv.shape), rdv) <= BWD_TOL
    assert perr(out, ref_out) <= PT_FWD_TOL
    if wl.name != "eq_single_neighbor":
        # (there every interior disc is the point itself: p = 1 and t = D, so dq and dk are exactly zero by cancellation;
        # fp32 leaves |t| 2^-24 ~ 1e-6 in their place, which the per-point measure would divide by its floor)
        assert max(perr(dq, rdq), perr(dk, rdk), perr(dv, rdv)) <= PT_BWD_TOL


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_benchmark_configurations_full_comparison(name):
    wl = WORKLOADS[name]
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)
    with _plan(wl) as plan:
        row_ptr, lat, off = plan.table()
        assert np.array_equal(row_ptr, g.row_ptr) and np.array_equal(lat, g.lat_in) and np.array_equal(off, g.lon_off)
        out, lse, dq, dk, dv = _run_gpu(plan, q, k, v, dout, True)
    ref_out = orc.forward(g, q, k, v)
    assert nerr(out.reshape(ref_out.shape), ref_out) <= FWD_TOL
    assert perr(out, ref_out) <= PT_FWD_TOL
    del ref_out
    rdq, rdk, rdv = orc.backward(g, q, k, v, dout)
    assert nerr(dq.reshape(rdq.shape), rdq) <= BWD_TOL
    assert nerr(dk.reshape(rdk.shape), rdk) <= BWD_TOL
    assert nerr(dv.reshape(rdv.shape), rdv) <= BWD_TOL
    assert max(perr(dq, rdq), perr(dk, rdk), perr(dv, rdv)) <= PT_BWD_TOL


@pytest.mark.parametrize("name, n_out, n_in", [("c3", 192, 96), ("c4", 160, 64), ("c5", 48, 12)])
def test_benchmark_configurations_sampled(name, n_out, n_in):
    """Full-size runs in the launch configuration the benchmark times; the oracle evaluates sampled points one
    by one.  The normalisation max|o| is taken over the sampled oracle values of each tensor."""
    wl = WORKLOADS[name]
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)
    with _plan(wl) as plan:
        assert plan.nnz == g.nnz
        out, lse, dq, dk, dv = _run_gpu(plan, q, k, v, dout, True)
    rng = np.random.default_rng(100 + wl.seed)
    po = sample_points(rng, wl.N, wl.nlat_out, wl.nlon_out, n_out)
    pi = sample_points(rng, wl.N, wl.nlat_in, wl.nlon_in, n_in)
    shape_o = (wl.N, wl.nlat_out, wl.nlon_out, wl.C)
    shape_i = (wl.N, wl.nlat_in, wl.nlon_in, wl.C)
    pick = lambda a, shape, p: a.reshape(shape)[p[:, 0], p[:, 1], p[:, 2]]
    assert nerr(pick(out, shape_o, po), orc.forward_points(g, q, k, v, po)) <= FWD_TOL
    assert nerr(pick(dq, shape_o, po), orc.dq_points(g, q, k, v, dout, po)) <= BWD_TOL
    rdk, rdv = orc.dkdv_points(g, q, k, v, dout, pi)
    assert nerr(pick(dk, shape_i, pi), rdk) <= BWD_TOL
    assert nerr(pick(dv, shape_i, pi), rdv) <= BWD_TOL
    # properties that hold at any size, over the whole tensors
    assert np.isfinite(out).all() and np.isfinite(dq).all() and np.isfinite(dk).all() and np.isfinite(dv).all()
    dv64, do64 = dv.reshape(shape_i).astype(np.float64), dout.reshape(shape_o).astype(np.float64)
    assert np.max(np.abs(dv64.sum((1, 2)) - do64.sum((1, 2)))) <= 1e-4 * np.max(np.abs(do64).sum((1, 2)))
    dk64 = dk.reshape(shape_i).astype(np.float64)
    assert np.max(np.abs(dk64.sum((1, 2)))) <= 1e-4 * np.max(np.abs(dk64).sum((1, 2)))


@pytest.mark.parametrize("q_scale, v_scale", [(12.0, 1.0), (1e-3, 50.0)], ids=["peaked_softmax", "flat_softmax_large_v"])
def test_extreme_score_magnitudes(q_scale, v_scale):
    """Scores of +-60 (softmax dominated by one neighbor; exp() overflows without the running maximum) and
    scores of ~1e-3 (flat softmax) with large values: no overflow, and the gates still hold."""
    wl = small_workload("extreme", 20, 64, 20, 64, EQ, EQ, 0.4, 1, 2, 32, 31)
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)
    q = (q * q_scale).astype(np.float32)
    v = (v * v_scale).astype(np.float32)
    with _plan(wl) as plan:
        out, lse, dq, dk, dv = _run_gpu(plan, q, k, v, dout, True)
    for a in (out, lse, dq, dk, dv):
        assert np.isfinite(a).all()
    ref_out = orc.forward(g, q, k, v)
    rdq, rdk, rdv = orc.backward(g, q, k, v, dout)
    assert nerr(out.reshape(ref_out.shape), ref_out) <= FWD_TOL
    assert nerr(dq.reshape(rdq.shape), rdq) <= BWD_TOL
    assert nerr(dk.reshape(rdk.shape), rdk) <= BWD_TOL
    assert nerr(dv.reshape(rdv.shape), rdv) <= BWD_TOL


LP_TOL = 5e-3   # stated tolerance of the reduced-precision variant (single TF32 product per contraction)


@pytest.mark.parametrize("wl", [SMALL[0], SMALL[2], SMALL[3], SMALL[15], SMALL[7], SMALL[10], SMALL[24], WORKLOADS["c2"]], ids=lambda w: w.name)
def test_reduced_precision_variant_against_oracle(wl):
    """sna_forward_tf32 / sna_backward_tf32: same operator, one TF32 product per contraction; its own, looser gate.  It must
    also be measurably less accurate than the default path (otherwise it is not the variant it claims to be)."""
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)
    with _plan(wl) as plan:
        qd, kd, vd, dd = _dev(q, k, v, dout)
        out, lse = plan.forward(qd, kd, vd, return_lse=True, precision="tf32")
        dq, dk, dv = plan.backward(qd, kd, vd, dd, out=out, lse=lse, precision="tf32")
        dq2, dk2, dv2 = plan.backward(qd, kd, vd, dd, precision="tf32")          # recomputed statistics
        torch.cuda.synchronize()
        sna.sna_plan_check(plan.handle)
    ref_out = orc.forward(g, q, k, v)
    rdq, rdk, rdv = orc.backward(g, q, k, v, dout)
    e_out = nerr(out.cpu().numpy().reshape(ref_out.shape), ref_out)
    assert 1e-5 < e_out <= LP_TOL
    for x, x2, r in ((dq, dq2, rdq), (dk, dk2, rdk), (dv, dv2, rdv)):
        assert nerr(x.cpu().numpy().reshape(r.shape), r) <= LP_TOL
        assert nerr(x2.cpu().numpy().reshape(r.shape), r) <= LP_TOL


def test_reduced_precision_variant_refuses_unsupported_shapes():
    wl = SMALL[5]      # C = 4: no tensor-core path
    q, k, v, dout = make_inputs(wl)
    with _plan(wl) as plan:
        qd, kd, vd = _dev(q, k, v)
        with pytest.raises(sna.SnaError) as e:
            plan.forward(qd, kd, vd, precision="tf32")
        assert e.value.status == sna.SNA_ERR_UNSUPPORTED
    torch.cuda.synchronize()


def test_global_limit_against_dense_oracle():
    wl = small_workload("global", 16, 32, 16, 32, EQ, EQ, math.pi, 1, 2, 32, 30)
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)
    with _plan(wl) as plan:
        out = plan.forward(*_dev(q, k, v)).cpu().numpy()
    ref = orc.dense_forward(np.repeat(g.omega, wl.nlon_in), q.reshape(wl.N, -1, wl.C), k.reshape(wl.N, -1, wl.C),
                            v.reshape(wl.N, -1, wl.C))
    assert nerr(out.reshape(ref.shape), ref) <= FWD_TOL


@pytest.mark.parametrize("shape", [(16, 32, 16, 32, EQ, EQ, 1, 2, 32), (33, 160, 17, 80, EQ, GL, 1, 2, 32),
                                   (40, 200, 40, 200, GL, GL, 2, 1, 32), (12, 24, 12, 24, EQ, EQ, 1, 2, 16),
                                   (20, 72, 20, 72, TZ, TZ, 1, 3, 32), (12, 24, 12, 24, TZ, EQ, 1, 2, 8)],
                         ids=["16x32", "33x160_down2", "40x200_gl", "C16_generic", "trapezoid", "trapezoid_C8_generic"])
@pytest.mark.parametrize("reuse", [True, False], ids=["saved_state", "recompute"])
def test_global_plan_against_oracle(shape, reuse):
    """sna_plan_create_global: forward against the dense definition written out, backward against the
    neighbourhood oracle with the cutoff at pi (whose forward the same dense definition pins on CPU)."""
    nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, B, H, C = shape
    wl = small_workload("global_plan", nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, math.pi, B, H, C, 31)
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)
    with sna.Plan(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, global_attention=True) as plan:
        out, lse, dq, dk, dv = _run_gpu(plan, q, k, v, dout, reuse)
        assert sna.sna_forward_kernel_count(plan.handle, C, True) == 1
    ref = orc.dense_forward(np.repeat(g.omega, wl.nlon_in), q.reshape(wl.N, -1, wl.C), k.reshape(wl.N, -1, wl.C),
                            v.reshape(wl.N, -1, wl.C))
    assert nerr(out.reshape(ref.shape), ref) <= FWD_TOL
    ref_out, ref_lse = orc.forward(g, q, k, v, return_lse=True)
    assert np.max(np.abs(lse.reshape(ref_lse.shape) - ref_lse)) <= 1e-4
    for name, x, r in zip(("dq", "dk", "dv"), (dq, dk, dv), orc.backward(g, q, k, v, dout)):
        assert nerr(x.reshape(r.shape), r) <= BWD_TOL, name
    if grid_in == TZ:       # the zero-weight pole ring: exact zeros, not small numbers
        assert not dk.reshape(wl.N, nlat_in, -1)[:, 0].any() and not dv.reshape(wl.N, nlat_in, -1)[:, 0].any()


def test_a_bounded_wait_that_runs_out_is_reported_once_and_the_plan_stays_usable():
    """The failure path of the bounded waits, without faulting or hanging anything: a probe kernel waits 1000 polls
    on a barrier nobody arrives on, gives up, records it; the check reports it once; compute calls still work."""
    wl = SMALL[0]
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)
    ref = orc.forward(g, q, k, v)
    with _plan(wl) as plan:
        sna.sna_plan_check(plan.handle)                          # clean to begin with
        sna.sna_debug_exercise_bounded_wait(plan.handle, 1000)
        with pytest.raises(sna.SnaError) as e:
            sna.sna_plan_check(plan.handle)
        assert e.value.status == sna.SNA_ERR_CUDA and "bounded wait" in str(e.value)
        sna.sna_plan_check(plan.handle)                          # reported once, then clear again
        out = plan.forward(*_dev(q, k, v))
        torch.cuda.synchronize()
        sna.sna_plan_check(plan.handle)
        assert nerr(out.cpu().numpy().reshape(ref.shape), ref) <= FWD_TOL
        with pytest.raises(sna.SnaError):
            sna.sna_debug_exercise_bounded_wait(plan.handle, 0)  # refused on the host


@pytest.mark.parametrize("wl", [SMALL[0], SMALL[2], SMALL[4], SMALL[6], SMALL[8], SMALL[26], WORKLOADS["c1"]], ids=lambda w: w.name)
def test_channels_first_entry_points_against_oracle(wl):
    """sna_forward_cf / sna_backward_cf: tensors [B, H*C, nlat, nlon]; the oracle sees the same values channels last."""
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)                               # [B, H, nlat, nlon, C]

    def to_cf(x):
        B, H, nlat, nlon, C = x.shape
        return np.ascontiguousarray(x.transpose(0, 1, 4, 2, 3).reshape(B, H * C, nlat, nlon))

    def to_cl(x, like):
        B, H, nlat, nlon, C = like.shape
        return x.reshape(B, H, C, nlat, nlon).transpose(0, 1, 3, 4, 2)

    with _plan(wl) as plan:
        out, state = plan.forward_cf(*_dev(to_cf(q), to_cf(k), to_cf(v)), heads=wl.H)
        dq, dk, dv = plan.backward_cf(_dev(to_cf(dout))[0], state, heads=wl.H)
        torch.cuda.synchronize()
        sna.sna_plan_check(plan.handle)
    ref_out = orc.forward(g, q, k, v)
    rdq, rdk, rdv = orc.backward(g, q, k, v, dout)
    assert nerr(to_cl(out.cpu().numpy(), q).reshape(ref_out.shape), ref_out) <= FWD_TOL
    assert nerr(to_cl(dq.cpu().numpy(), q).reshape(rdq.shape), rdq) <= BWD_TOL
    assert nerr(to_cl(dk.cpu().numpy(), k).reshape(rdk.shape), rdk) <= BWD_TOL
    assert nerr(to_cl(dv.cpu().numpy(), k).reshape(rdv.shape), rdv) <= BWD_TOL


def test_channels_first_autograd_wrapper_and_buffer_checks():
    from paper_2505_11157_b200.autograd import spherical_neighborhood_attention_cf
    wl = SMALL[0]
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)
    cf = lambda x: torch.from_numpy(np.ascontiguousarray(x.transpose(0, 1, 4, 2, 3).reshape(x.shape[0], -1, x.shape[2], x.shape[3]))).cuda()
    with _plan(wl) as plan:
        qt, kt, vt = (cf(x).requires_grad_(True) for x in (q, k, v))
        out = spherical_neighborhood_attention_cf(plan, qt, kt, vt, heads=wl.H)
        out.backward(cf(dout))
        torch.cuda.synchronize()
        rdq, rdk, rdv = orc.backward(g, q, k, v, dout)
        back = lambda t, like: t.detach().cpu().numpy().reshape(like.shape[0], like.shape[1], like.shape[4], like.shape[2], like.shape[3]).transpose(0, 1, 3, 4, 2)
        assert nerr(back(qt.grad, q).reshape(rdq.shape), rdq) <= BWD_TOL
        assert nerr(back(kt.grad, k).reshape(rdk.shape), rdk) <= BWD_TOL
        assert nerr(back(vt.grad, k).reshape(rdv.shape), rdv) <= BWD_TOL
        # a state buffer that is too small is refused on the host
        small = torch.empty(256, dtype=torch.uint8, device="cuda")
        with pytest.raises(sna.SnaError) as e:
            plan.forward_cf(cf(q), cf(k), cf(v), heads=wl.H, state=small)
        assert e.value.status == sna.SNA_ERR_WORKSPACE
        with pytest.raises(ValueError):
            plan.forward_cf(cf(q), cf(k), cf(v), heads=5)     # channel count not divisible by the heads
    torch.cuda.synchronize()


def _random_problems(count, seed):
    """Seeded random problems that the oracle accepts; wide rings so that banded, wide and whole-ring windows all occur."""
    rng = np.random.default_rng(seed)
    found = []
    while len(found) < count:
        ps = int(rng.choice([1, 1, 2, 2, 3, 4]))
        nlon_out = int(rng.integers(32, 200 // ps + 33))
        nlat_in, nlat_out = int(rng.integers(6, 25)), int(rng.integers(6, 25))
        gi, go = int(rng.integers(0, 3)), int(rng.integers(0, 3))
        theta = float(rng.uniform(0.25, 1.3))
        C = int(rng.choice([32, 32, 32, 16, 64, 8]))
        wl = small_workload(f"random{len(found)}", nlat_in, nlon_out * ps, nlat_out, nlon_out, gi, go, theta, 1, int(rng.integers(1, 3)), C,
                            100 + len(found))
        try:
            _geometry(wl)
        except orc.OracleError:
            continue
        found.append(wl)
    return found


@pytest.mark.parametrize("wl", _random_problems(12, 11157), ids=lambda w: f"{w.name}_{w.nlat_in}x{w.nlon_in}_to_{w.nlat_out}x{w.nlon_out}_C{w.C}")
def test_random_problems_full_comparison(wl):
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)
    with _plan(wl) as plan:
        out, lse, dq, dk, dv = _run_gpu(plan, q, k, v, dout, True)
    ref_out = orc.forward(g, q, k, v)
    rdq, rdk, rdv = orc.backward(g, q, k, v, dout)
    assert nerr(out.reshape(ref_out.shape), ref_out) <= FWD_TOL
    for name, x, r in zip(("dq", "dk", "dv"), (dq, dk, dv), (rdq, rdk, rdv)):
        assert nerr(x.reshape(r.shape), r) <= BWD_TOL, name
    assert perr(out, ref_out) <= PT_FWD_TOL


def test_multi_head_module_matches_oracle_composition():
    """The nn.Module wrapper: pointwise projections (library GEMMs) around the channels-first operator.  Reference:
    the same projections in fp64 numpy around the oracle; gradients of the projection weights through autograd."""
    from paper_2505_11157_b200.module import SphericalNeighborhoodAttention
    nlat_in, nlon_in, nlat_out, nlon_out, heads, hd, cin = 17, 48, 9, 24, 2, 16, 12
    g = orc.geometry(nlat_in, nlon_in, nlat_out, nlon_out, EQ, EQ, 0.6)
    torch.manual_seed(5)
    with sna.Plan(nlat_in, nlon_in, nlat_out, nlon_out, EQ, EQ, 0.6) as plan:
        layer = SphericalNeighborhoodAttention(plan, cin, heads, hd).cuda()
        prev = torch.backends.cudnn.allow_tf32, torch.backends.cuda.matmul.allow_tf32
        torch.backends.cudnn.allow_tf32 = torch.backends.cuda.matmul.allow_tf32 = False
        try:
            xq = torch.randn(2, cin, nlat_out, nlon_out, device="cuda", requires_grad=True)
            xkv = torch.randn(2, cin, nlat_in, nlon_in, device="cuda", requires_grad=True)
            y = layer(xq, xkv)
            y.square().sum().backward()
            torch.cuda.synchronize()
        finally:
            torch.backends.cudnn.allow_tf32, torch.backends.cuda.matmul.allow_tf32 = prev
    f64 = lambda t: t.detach().cpu().double().numpy()
    proj = lambda x, w, b: np.einsum("oi,bihw->bohw", f64(w)[:, :, 0, 0], x) + f64(b)[None, :, None, None]
    heads_last = lambda t: t.reshape(t.shape[0], heads, hd, t.shape[2], t.shape[3]).transpose(0, 1, 3, 4, 2)   # [B, H, lat, lon, C]
    q, k, v = (heads_last(proj(f64(x), w, b)) for x, w, b in ((xq, layer.wq, layer.bq), (xkv, layer.wk, layer.bk), (xkv, layer.wv, layer.bv)))
    att = orc.forward(g, q, k, v).reshape(2, heads, nlat_out, nlon_out, hd).transpose(0, 1, 4, 2, 3).reshape(2, heads * hd, nlat_out, nlon_out)
    ref = proj(att, layer.wo, layer.bo)
    assert nerr(f64(y), ref) <= 2e-5
    assert all(p.grad is not None and torch.isfinite(p.grad).all() for p in layer.parameters())
    assert xq.grad is not None and xkv.grad is not None and float(xkv.grad.abs().max()) > 0


def test_results_are_reproducible_bit_for_bit():
    wl = SMALL[2]
    q, k, v, dout = make_inputs(wl)
    with _plan(wl) as plan:
        a = _run_gpu(plan, q, k, v, dout, True)
        b = _run_gpu(plan, q, k, v, dout, True)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


@pytest.mark.parametrize("name, runs", [("c2", 12), ("c3", 12), ("c4", 8), ("c5", 12)])
def test_benchmark_configurations_are_reproducible_bit_for_bit(name, runs):
    """Every sum is taken in a fixed order, so repeated runs must agree bit for bit at full size too.  This is also the
    sharpest detector of a race between the roles of the pipelined kernels: a stale operand or an early read changes
    some 32-row block of some tile in some run (it caught a second arrival counted into the wrong barrier phase and
    an early reuse of the staging tiles)."""
    wl = WORKLOADS[name]
    qd, kd, vd, dd = _dev(*make_inputs(wl))
    with _plan(wl) as plan:
        first = None
        for run in range(runs):
            out, lse = plan.forward(qd, kd, vd, return_lse=True)
            dq, dk, dv = plan.backward(qd, kd, vd, dd, out=out, lse=lse)
            torch.cuda.synchronize()
            if first is None:
                first = [t.clone() for t in (out, lse, dq, dk, dv)]
            else:
                for tname, a, b in zip(("out", "lse", "dq", "dk", "dv"), (out, lse, dq, dk, dv), first):
                    assert torch.equal(a, b), (name, run, tname)
        sna.sna_plan_check(plan.handle)


def test_longitude_roll_equivariance_on_gpu():
    wl = SMALL[2]
    q, k, v, dout = make_inputs(wl)
    ps, s = wl.nlon_in // wl.nlon_out, 5
    with _plan(wl) as plan:
        out, _, dq, dk, dv = _run_gpu(plan, q, k, v, dout)
        r_o = lambda a: np.ascontiguousarray(np.roll(a, s, axis=3))
        r_i = lambda a: np.ascontiguousarray(np.roll(a, s * ps, axis=3))
        out2, _, dq2, dk2, dv2 = _run_gpu(plan, r_o(q), r_i(k), r_i(v), r_o(dout))
    for a, b, roll in ((out, out2, r_o), (dq, dq2, r_o), (dk, dk2, r_i), (dv, dv2, r_i)):
        assert np.max(np.abs(roll(a) - b)) <= 2e-5 * np.max(np.abs(a))


def test_argument_errors_launch_nothing():
    wl = SMALL[0]
    q, k, v, dout = make_inputs(wl)
    with _plan(wl) as plan:
        qd, kd, vd, dd = _dev(q, k, v, dout)
        out = torch.empty_like(qd)
        with pytest.raises(sna.SnaError) as e:
            sna.sna_forward(plan.handle, qd, kd, vd, out, wl.B, wl.H, 6)
        assert e.value.status == sna.SNA_ERR_UNSUPPORTED
        with pytest.raises(sna.SnaError) as e:
            sna.sna_forward(plan.handle, qd.data_ptr() + 4, kd, vd, out, wl.B, wl.H, wl.C)
        assert e.value.status == sna.SNA_ERR_INVALID_ARG
        with pytest.raises(sna.SnaError) as e:
            sna.sna_forward(plan.handle, None, kd, vd, out, wl.B, wl.H, wl.C)
        assert e.value.status == sna.SNA_ERR_INVALID_ARG
        ws = torch.empty(256, dtype=torch.uint8, device="cuda")
        with pytest.raises(sna.SnaError) as e:
            sna.sna_backward_ex(plan.handle, qd, kd, vd, dd, None, None, torch.empty_like(qd), torch.empty_like(kd),
                                torch.empty_like(kd), ws, ws.numel(), wl.B, wl.H, wl.C)
        assert e.value.status == sna.SNA_ERR_WORKSPACE
        torch.cuda.synchronize()


def test_call_with_another_device_current_is_refused_on_the_host():
    """A plan belongs to the device it was created on.  With another device current the call must fail validation
    (the check runs on the host before any launch), not launch with the first device's addresses."""
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two visible GPUs")
    wl = SMALL[0]
    q, k, v, dout = make_inputs(wl)
    with torch.cuda.device(0):
        plan = _plan(wl)
        qd, kd, vd, dd = _dev(q, k, v, dout)
        out = torch.empty_like(qd)
    try:
        with torch.cuda.device(1):
            with pytest.raises(sna.SnaError) as e:
                sna.sna_forward(plan.handle, qd, kd, vd, out, wl.B, wl.H, wl.C, stream=0)
            assert e.value.status == sna.SNA_ERR_INVALID_ARG
            with pytest.raises(sna.SnaError) as e:
                sna.sna_backward_static(plan.handle, qd, kd, vd, dd, out, torch.empty_like(kd), torch.empty_like(kd),
                                        wl.B, wl.H, wl.C, stream=0)
            assert e.value.status == sna.SNA_ERR_INVALID_ARG
    finally:
        with torch.cuda.device(0):
            plan.close()


def test_fp32_fma_peak_probe_is_plausible():
    props = torch.cuda.get_device_properties(0)
    nominal = props.multi_processor_count * 128 * 2 * 1.965e9 / 1e12      # B200: 148 SMs -> 74.4 TFLOP/s
    measured = sna.sna_measure_fp32_fma_peak()
    assert 0.5 * nominal < measured < 1.1 * nominal


def test_autograd_wrapper_matches_oracle_gradients():
    from paper_2505_11157_b200.autograd import spherical_neighborhood_attention
    wl = SMALL[2]
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)
    with _plan(wl) as plan:
        qd, kd, vd, dd = _dev(q, k, v, dout)
        for t in (qd, kd, vd):
            t.requires_grad_(True)
        out = spherical_neighborhood_attention(plan, qd, kd, vd)
        (out * dd).sum().backward()
        torch.cuda.synchronize()
        got = [t.grad.cpu().numpy() for t in (qd, kd, vd)]
    refs = orc.backward(g, q, k, v, dout)
    for x, r in zip(got, refs):
        assert nerr(x.reshape(r.shape), r) <= BWD_TOL


def test_runs_on_a_side_stream():
    wl = SMALL[0]
    g = _geometry(wl)
    q, k, v, dout = make_inputs(wl)
    ref = orc.forward(g, q, k, v)
    stream = torch.cuda.Stream()
    with _plan(wl) as plan:
        with torch.cuda.stream(stream):
            qd, kd, vd = _dev(q, k, v)
            out = plan.forward(qd, kd, vd, stream=stream)
        stream.synchronize()
    assert nerr(out.cpu().numpy().reshape(ref.shape), ref) <= FWD_TOL
