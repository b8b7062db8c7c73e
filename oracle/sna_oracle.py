"""ctypes front end of the fp64 CPU oracle (``sna_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the CPU-baseline / reference
legs of the benchmark.  The CUDA library and its Python binding never import this module, and this
module never imports them.

The wrapper only marshals arguments: inputs are widened to float64 (exactly, when they are float32)
and every result comes back as float64.  The arithmetic lives in the C file, whose header lists the
passages of the paper each routine follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sna_oracle.c")
_LIB = os.path.join(_HERE, "libsna_oracle.so")

EQUIANGULAR = 0
LEGENDRE_GAUSS = 1
EQUIANGULAR_TRAPEZOID = 2   # the grid App. A.1 prints: theta_i = pi i / nlat, weights ~ sin(theta_i), pole ring weight 0

_ERRORS = {1: "invalid argument", 2: "ambiguous tie on the disc boundary", 3: "empty neighborhood",
           4: "capacity too small"}


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle error {code}: {_ERRORS.get(code, '?')}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (nothing else) if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-Wall",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _check(rc: int):
    if rc != 0:
        raise OracleError(rc)


def _dp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _i64p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))


def _i32p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def _f64(a):
    return np.ascontiguousarray(np.asarray(a), dtype=np.float64)


def num_threads() -> int:
    return int(_load().sna_oracle_num_threads())


def colatitudes(grid: int, nlat: int) -> np.ndarray:
    th = np.empty(nlat, dtype=np.float64)
    _check(_load().sna_oracle_colatitudes(grid, nlat, _dp(th)))
    return th


def latitude_weights(grid: int, nlat: int) -> np.ndarray:
    w = np.empty(nlat, dtype=np.float64)
    _check(_load().sna_oracle_latitude_weights(grid, nlat, _dp(w)))
    return w


def quad_weights(grid: int, nlat: int, nlon: int) -> np.ndarray:
    w = np.empty(nlat, dtype=np.float64)
    _check(_load().sna_oracle_quad_weights(grid, nlat, nlon, _dp(w)))
    return w


@dataclass
class Geometry:
    """Grids, per-ring point weights and the brute-force neighborhood table of one problem."""
    nlat_in: int
    nlon_in: int
    nlat_out: int
    nlon_out: int
    grid_in: int
    grid_out: int
    theta_cutoff: float
    row_ptr: np.ndarray   # int64 [nlat_out + 1]
    lat_in: np.ndarray    # int32 [nnz]
    lon_off: np.ndarray   # int32 [nnz], in [0, nlon_in)
    omega: np.ndarray     # float64 [nlat_in]

    @property
    def nnz(self) -> int:
        return int(self.row_ptr[-1])


def geometry(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, theta_cutoff) -> Geometry:
    if nlon_out < 1 or nlon_in % nlon_out != 0:
        raise OracleError(1)
    lib = _load()
    nnz = ctypes.c_int64(0)
    row_ptr = np.zeros(nlat_out + 1, dtype=np.int64)
    _check(lib.sna_oracle_neighborhood(grid_in, nlat_in, nlon_in, grid_out, nlat_out,
                                       ctypes.c_double(theta_cutoff), _i64p(row_ptr), None, None,
                                       ctypes.c_int64(0), ctypes.byref(nnz)))
    lat = np.empty(nnz.value, dtype=np.int32)
    off = np.empty(nnz.value, dtype=np.int32)
    _check(lib.sna_oracle_neighborhood(grid_in, nlat_in, nlon_in, grid_out, nlat_out,
                                       ctypes.c_double(theta_cutoff), _i64p(row_ptr), _i32p(lat), _i32p(off),
                                       ctypes.c_int64(nnz.value), ctypes.byref(nnz)))
    return Geometry(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, float(theta_cutoff),
                    row_ptr, lat, off, quad_weights(grid_in, nlat_in, nlon_in))


def _geom_args(g: Geometry):
    return (g.nlat_in, g.nlon_in, g.nlat_out, g.nlon_out, _i64p(g.row_ptr), _i32p(g.lat_in), _i32p(g.lon_off),
            _dp(g.omega))


def _shapes(g: Geometry, q, k):
    q = _f64(q)
    k = _f64(k)
    C = q.shape[-1]
    N = q.size // (g.nlat_out * g.nlon_out * C)
    assert q.size == N * g.nlat_out * g.nlon_out * C
    assert k.size == N * g.nlat_in * g.nlon_in * C, "k has the wrong number of elements"
    return q, k, N, C


def forward(g: Geometry, q, k, v, return_lse: bool = False):
    """out (float64, shaped like q) and optionally lse = max + log(sum) per output point."""
    q, k, N, C = _shapes(g, q, k)
    v = _f64(v)
    out = np.empty_like(q)
    lse = np.empty(q.shape[:-1], dtype=np.float64)
    _check(_load().sna_oracle_forward(*_geom_args(g), N, C, _dp(q), _dp(k), _dp(v), _dp(out), _dp(lse)))
    return (out, lse) if return_lse else out


def backward(g: Geometry, q, k, v, dout):
    """(dq, dk, dv) in float64."""
    q, k, N, C = _shapes(g, q, k)
    v = _f64(v)
    dout = _f64(dout)
    dq = np.empty_like(q)
    dk = np.empty_like(k)
    dv = np.empty_like(k)
    _check(_load().sna_oracle_backward(*_geom_args(g), N, C, _dp(q), _dp(k), _dp(v), _dp(dout),
                                       _dp(dq), _dp(dk), _dp(dv)))
    return dq, dk, dv


def _points(pts):
    pts = np.ascontiguousarray(np.asarray(pts), dtype=np.int32)
    assert pts.ndim == 2 and pts.shape[1] == 3
    return pts


def forward_points(g: Geometry, q, k, v, pts):
    """Forward at output points pts[:, (n, h, w)] -> [npts, C]."""
    q, k, N, C = _shapes(g, q, k)
    v = _f64(v)
    pts = _points(pts)
    out = np.empty((pts.shape[0], C), dtype=np.float64)
    _check(_load().sna_oracle_forward_points(*_geom_args(g), N, C, _dp(q), _dp(k), _dp(v),
                                             ctypes.c_int64(pts.shape[0]), _i32p(pts), _dp(out)))
    return out


def dq_points(g: Geometry, q, k, v, dout, pts):
    q, k, N, C = _shapes(g, q, k)
    v = _f64(v)
    dout = _f64(dout)
    pts = _points(pts)
    dq = np.empty((pts.shape[0], C), dtype=np.float64)
    _check(_load().sna_oracle_dq_points(*_geom_args(g), N, C, _dp(q), _dp(k), _dp(v), _dp(dout),
                                        ctypes.c_int64(pts.shape[0]), _i32p(pts), _dp(dq)))
    return dq


def dkdv_points(g: Geometry, q, k, v, dout, pts):
    """dk, dv at input points pts[:, (n, h', w')] -> two [npts, C] arrays."""
    q, k, N, C = _shapes(g, q, k)
    v = _f64(v)
    dout = _f64(dout)
    pts = _points(pts)
    dk = np.empty((pts.shape[0], C), dtype=np.float64)
    dv = np.empty((pts.shape[0], C), dtype=np.float64)
    _check(_load().sna_oracle_dkdv_points(*_geom_args(g), N, C, _dp(q), _dp(k), _dp(v), _dp(dout),
                                          ctypes.c_int64(pts.shape[0]), _i32p(pts), _dp(dk), _dp(dv)))
    return dk, dv


def dense_forward(wpt, q, k, v):
    """Dense weighted attention over all input points: q [N, Mout, C], k/v [N, Min, C], wpt [Min]."""
    q = _f64(q)
    k = _f64(k)
    v = _f64(v)
    wpt = _f64(wpt)
    N, Mout, C = q.shape
    Min = k.shape[1]
    assert wpt.shape == (Min,)
    out = np.empty_like(q)
    _check(_load().sna_oracle_dense_forward(N, ctypes.c_int64(Mout), ctypes.c_int64(Min), C, _dp(wpt),
                                            _dp(q), _dp(k), _dp(v), _dp(out)))
    return out
