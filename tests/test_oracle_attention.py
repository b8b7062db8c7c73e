"""Pins for the oracle's forward and backward passes.

Forward: Eq. (s2_attention_discrete_detailed); backward: App. B.4.  The pins are what the paper and the
mathematics fix: normalisation of the attention weights, the role of the quadrature weights in numerator
and denominator, longitude-roll equivariance (the table does not depend on the output longitude), the
global limit theta_cutoff = pi computed by a library dense attention with additive mask log(w)
(App. B.2), and finite differences.
"""
import math

import numpy as np
import pytest
import torch

from oracle import sna_oracle as orc

EQ, GL, TZ = orc.EQUIANGULAR, orc.LEGENDRE_GAUSS, orc.EQUIANGULAR_TRAPEZOID


def _rand(g, N, C, seed, dtype=np.float64):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((N, g.nlat_out, g.nlon_out, C)).astype(dtype)
    k = rng.standard_normal((N, g.nlat_in, g.nlon_in, C)).astype(dtype)
    v = rng.standard_normal((N, g.nlat_in, g.nlon_in, C)).astype(dtype)
    dout = rng.standard_normal((N, g.nlat_out, g.nlon_out, C)).astype(dtype)
    return q, k, v, dout


GEOMS = {
    "eq_same": (12, 24, 12, 24, EQ, EQ, 0.6),
    "eq_down": (17, 32, 9, 16, EQ, EQ, 0.5),
    "gl_same": (10, 20, 10, 20, GL, GL, 0.7),
    "gl_to_eq_down3": (12, 24, 7, 8, GL, EQ, 0.8),
    "tz_same": (12, 24, 12, 24, TZ, TZ, 0.6),
    "tz_down": (16, 32, 8, 16, TZ, TZ, 0.5),
}


@pytest.fixture(scope="module", params=list(GEOMS))
def geom(request):
    return orc.geometry(*GEOMS[request.param])


def test_constant_v_gives_constant_output(geom):
    q, k, v, _ = _rand(geom, 2, 8, 0)
    v[...] = np.arange(8)[None, None, None, :] * 0.5 - 1.0
    out = orc.forward(geom, q, k, v)
    assert np.allclose(out, v[:, :1, :1, :], rtol=0, atol=1e-14)


def test_zero_q_gives_quadrature_weighted_neighborhood_mean(geom):
    # with q = 0 every exp() is 1, so out_i = sum_j w_j v_j / sum_j w_j over the disc: the weights must
    # appear in numerator and denominator
    q, k, v, _ = _rand(geom, 1, 4, 1)
    q[...] = 0
    out = orc.forward(geom, q, k, v)
    ps = geom.nlon_in // geom.nlon_out
    rng = np.random.default_rng(5)
    for _ in range(12):
        h, w = int(rng.integers(geom.nlat_out)), int(rng.integers(geom.nlon_out))
        lat = geom.lat_in[geom.row_ptr[h]:geom.row_ptr[h + 1]]
        col = (geom.lon_off[geom.row_ptr[h]:geom.row_ptr[h + 1]] + w * ps) % geom.nlon_in
        wts = geom.omega[lat]
        expect = (wts[:, None] * v[0, lat, col, :]).sum(0) / wts.sum()
        assert np.allclose(out[0, h, w], expect, rtol=0, atol=1e-14)
    # the result must differ from the unweighted mean (otherwise the pin would not see a dropped weight)
    h = 1
    lat = geom.lat_in[geom.row_ptr[h]:geom.row_ptr[h + 1]]
    col = geom.lon_off[geom.row_ptr[h]:geom.row_ptr[h + 1]] % geom.nlon_in
    assert not np.allclose(out[0, h, 0], v[0, lat, col, :].mean(0), atol=1e-6)


def test_constant_k_behaves_like_zero_q(geom):
    q, k, v, _ = _rand(geom, 1, 4, 2)
    k[...] = np.array([0.3, -1.0, 2.0, 0.5])
    out = orc.forward(geom, q, k, v)
    out0 = orc.forward(geom, np.zeros_like(q), k, v)
    assert np.allclose(out, out0, rtol=0, atol=1e-13)


def test_adding_a_constant_vector_to_every_k_changes_nothing(geom):
    q, k, v, _ = _rand(geom, 2, 4, 3)
    out = orc.forward(geom, q, k, v)
    out2 = orc.forward(geom, q, k + np.array([1.0, -2.0, 0.5, 3.0]), v)
    assert np.allclose(out, out2, rtol=0, atol=1e-12)


def test_longitude_roll_equivariance(geom):
    q, k, v, dout = _rand(geom, 2, 4, 4)
    ps = geom.nlon_in // geom.nlon_out
    out = orc.forward(geom, q, k, v)
    dq, dk, dv = orc.backward(geom, q, k, v, dout)
    s = 3
    r_out = lambda a: np.roll(a, s, axis=2)
    r_in = lambda a: np.roll(a, s * ps, axis=2)
    out_r = orc.forward(geom, r_out(q), r_in(k), r_in(v))
    assert np.allclose(out_r, r_out(out), rtol=0, atol=1e-14)
    dq_r, dk_r, dv_r = orc.backward(geom, r_out(q), r_in(k), r_in(v), r_out(dout))
    assert np.allclose(dq_r, r_out(dq), rtol=0, atol=1e-13)
    assert np.allclose(dk_r, r_in(dk), rtol=0, atol=1e-13)
    assert np.allclose(dv_r, r_in(dv), rtol=0, atol=1e-13)


def test_tiny_cutoff_copies_v():
    # same grid: out(h, w) = v(h, w) away from the poles
    g = orc.geometry(9, 16, 9, 16, EQ, EQ, 0.05)
    q, k, v, _ = _rand(g, 1, 4, 6)
    out = orc.forward(g, q, k, v)
    assert np.allclose(out[:, 1:-1], v[:, 1:-1], rtol=0, atol=1e-14)
    # nested grids, half the resolution: out(h, w) = v(2h, 2w); catches a wrong shift direction or stride
    g = orc.geometry(17, 32, 9, 16, EQ, EQ, 0.05)
    q, k, v, _ = _rand(g, 1, 4, 7)
    out = orc.forward(g, q, k, v)
    assert np.allclose(out[:, 1:-1], v[:, 2:-2:2, ::2], rtol=0, atol=1e-14)


def _sdpa(q, k, v, omega_pt):
    """Library dense attention with additive mask log(w) (App. B.2); fp64, CPU."""
    N, Mo, C = q.shape
    mask = torch.log(torch.from_numpy(omega_pt))[None, None, :].expand(N, Mo, -1)
    return torch.nn.functional.scaled_dot_product_attention(q_t := torch.from_numpy(q).requires_grad_(True),
                                                            k_t := torch.from_numpy(k).requires_grad_(True),
                                                            v_t := torch.from_numpy(v).requires_grad_(True),
                                                            attn_mask=mask), (q_t, k_t, v_t)


@pytest.mark.parametrize("args", [(8, 16, 8, 16, EQ, EQ), (9, 12, 5, 6, EQ, GL), (6, 12, 6, 12, GL, GL), (8, 16, 8, 16, TZ, TZ)])
def test_global_limit_matches_library_dense_attention(args):
    g = orc.geometry(*args, math.pi)
    N, C = 2, 8
    q, k, v, dout = _rand(g, N, C, 8)
    omega_pt = np.repeat(g.omega, g.nlon_in)
    qf, kf, vf = q.reshape(N, -1, C), k.reshape(N, -1, C), v.reshape(N, -1, C)
    ref, (qt, kt, vt) = _sdpa(qf, kf, vf, omega_pt)
    out = orc.forward(g, q, k, v)
    assert np.allclose(out.reshape(N, -1, C), ref.detach().numpy(), rtol=0, atol=1e-13)
    # dense oracle routine (no table) agrees too
    assert np.allclose(orc.dense_forward(omega_pt, qf, kf, vf), ref.detach().numpy(), rtol=0, atol=1e-13)
    # gradients through the library routine
    ref.backward(torch.from_numpy(dout.reshape(N, -1, C)))
    dq, dk, dv = orc.backward(g, q, k, v, dout)
    assert np.allclose(dq.reshape(N, -1, C), qt.grad.numpy(), rtol=0, atol=1e-12)
    assert np.allclose(dk.reshape(N, -1, C), kt.grad.numpy(), rtol=0, atol=1e-12)
    assert np.allclose(dv.reshape(N, -1, C), vt.grad.numpy(), rtol=0, atol=1e-12)


def test_zero_weight_pole_ring_contributes_nothing():
    # on the grid of Eq. (latlon_grid) the pole ring has quadrature weight sin(0) = 0: its points are inside the
    # discs near the pole but neither their keys nor their values can reach any output, and they get no gradient
    g = orc.geometry(10, 20, 10, 20, TZ, TZ, 0.7)
    assert g.omega[0] == 0.0 and np.any(g.lat_in == 0)
    q, k, v, dout = _rand(g, 2, 6, 21)
    out = orc.forward(g, q, k, v)
    k2, v2 = k.copy(), v.copy()
    k2[:, 0] += 3.0
    v2[:, 0] = 100.0
    # (not bit-equal: a pole-ring score may set the running maximum, which moves the rounding)
    assert np.allclose(orc.forward(g, q, k2, v2), out, rtol=0, atol=1e-13)
    dq, dk, dv = orc.backward(g, q, k, v, dout)
    assert not dk[:, 0].any() and not dv[:, 0].any()
    assert dk[:, 1].any() and dv[:, 1].any() and np.isfinite(dq).all()


def test_a_disc_of_total_weight_zero_is_reported():
    # the disc of the pole output point holds only the (zero-weight) pole ring: Eq. (s2_attention_discrete_detailed) is 0/0
    with pytest.raises(orc.OracleError) as e:
        orc.geometry(16, 32, 16, 32, TZ, TZ, 0.05)
    assert e.value.code == 3
    orc.geometry(16, 32, 16, 32, TZ, TZ, 0.25)      # one more ring inside: defined again


def test_lse_definition(geom):
    q, k, v, _ = _rand(geom, 1, 4, 9)
    out, lse = orc.forward(geom, q, k, v, return_lse=True)
    h, w = geom.nlat_out // 2, 1
    ps = geom.nlon_in // geom.nlon_out
    lat = geom.lat_in[geom.row_ptr[h]:geom.row_ptr[h + 1]]
    col = (geom.lon_off[geom.row_ptr[h]:geom.row_ptr[h + 1]] + w * ps) % geom.nlon_in
    s = (k[0, lat, col, :] @ q[0, h, w]) / 2.0
    assert abs(lse[0, h, w] - math.log(np.sum(np.exp(s) * geom.omega[lat]))) < 1e-13


@pytest.mark.parametrize("args", [(6, 12, 6, 12, EQ, EQ, 0.9), (8, 16, 4, 8, EQ, EQ, 0.9), (5, 10, 5, 10, GL, GL, 1.0),
                                  (6, 12, 6, 12, TZ, TZ, 0.9)])
def test_backward_matches_central_finite_differences(args):
    g = orc.geometry(*args)
    N, C = 1, 4
    q, k, v, dout = _rand(g, N, C, 10)
    dq, dk, dv = orc.backward(g, q, k, v, dout)
    loss = lambda q_, k_, v_: float(np.sum(orc.forward(g, q_, k_, v_) * dout))
    rng = np.random.default_rng(11)
    eps = 1e-6
    for name, arr, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        flat = arr.reshape(-1)
        for idx in rng.choice(flat.size, 20, replace=False):
            old = flat[idx]
            flat[idx] = old + eps
            lp = loss(q, k, v)
            flat[idx] = old - eps
            lm = loss(q, k, v)
            flat[idx] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - grad.reshape(-1)[idx]) < 2e-8 * max(1.0, abs(fd)), (name, idx, fd, grad.reshape(-1)[idx])


def test_backward_invariants(geom):
    N, C = 2, 4
    q, k, v, dout = _rand(geom, N, C, 12)
    dq, dk, dv = orc.backward(geom, q, k, v, dout)
    # sum_j dv_j = sum_i dy_i (attention weights sum to one), per slice and channel
    assert np.allclose(dv.sum((1, 2)), dout.sum((1, 2)), rtol=0, atol=1e-12)
    # shifting every k by a constant changes nothing => sum_j dk_j = 0
    assert np.allclose(dk.sum((1, 2)), 0, atol=1e-12)
    # scores are bilinear: sum_i q_i.dq_i = sum_j k_j.dk_j
    assert np.allclose((q * dq).sum((1, 2, 3)), (k * dk).sum((1, 2, 3)), rtol=0, atol=1e-11)


def test_point_routines_agree_with_full_routines(geom):
    N, C = 2, 4
    q, k, v, dout = _rand(geom, N, C, 13)
    out = orc.forward(geom, q, k, v)
    dq, dk, dv = orc.backward(geom, q, k, v, dout)
    rng = np.random.default_rng(14)
    po = np.stack([rng.integers(0, N, 16), rng.integers(0, geom.nlat_out, 16), rng.integers(0, geom.nlon_out, 16)], 1)
    pi = np.stack([rng.integers(0, N, 16), rng.integers(0, geom.nlat_in, 16), rng.integers(0, geom.nlon_in, 16)], 1)
    po[0, 1], pi[0, 1], pi[1, 1] = 0, 0, geom.nlat_in - 1
    assert np.allclose(orc.forward_points(geom, q, k, v, po), out[po[:, 0], po[:, 1], po[:, 2]], rtol=0, atol=1e-14)
    assert np.allclose(orc.dq_points(geom, q, k, v, dout, po), dq[po[:, 0], po[:, 1], po[:, 2]], rtol=0, atol=1e-14)
    dkp, dvp = orc.dkdv_points(geom, q, k, v, dout, pi)
    assert np.allclose(dkp, dk[pi[:, 0], pi[:, 1], pi[:, 2]], rtol=0, atol=1e-13)
    assert np.allclose(dvp, dv[pi[:, 0], pi[:, 1], pi[:, 2]], rtol=0, atol=1e-13)


def test_float32_inputs_are_widened_exactly():
    g = orc.geometry(6, 12, 6, 12, EQ, EQ, 0.9)
    q, k, v, _ = _rand(g, 1, 4, 15, dtype=np.float32)
    a = orc.forward(g, q, k, v)
    b = orc.forward(g, q.astype(np.float64), k.astype(np.float64), v.astype(np.float64))
    assert a.dtype == np.float64 and np.array_equal(a, b)
