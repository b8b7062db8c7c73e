"""Seeded synthetic workloads shaped like the paper's (Sec. 4 and App. C.1: 128x256 and 256x512
equiangular panoramas, Gaussian-grid fields, latent width 128 split into heads, cutoffs of a few
grid spacings).  They stand in for the paper's datasets, which are not needed: the cost of the
operator does not depend on the values.

This module holds no arithmetic of the method.  It only names the five benchmark configurations and
draws i.i.d. normal tensors on the host with numpy's PCG64, in the fixed order q, k, v, dout, so the
CPU oracle and the CUDA path can be fed the very same arrays.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

EQUIANGULAR = 0
LEGENDRE_GAUSS = 1


@dataclass(frozen=True)
class Workload:
    name: str
    nlat_in: int
    nlon_in: int
    nlat_out: int
    nlon_out: int
    grid_in: int
    grid_out: int
    theta_cutoff: float
    B: int
    H: int
    C: int
    seed: int
    dout_std: float = 1.0
    description: str = ""

    @property
    def N(self) -> int:
        return self.B * self.H

    @property
    def q_shape(self):
        return (self.B, self.H, self.nlat_out, self.nlon_out, self.C)

    @property
    def k_shape(self):
        return (self.B, self.H, self.nlat_in, self.nlon_in, self.C)


WORKLOADS = {
    "c1": Workload("c1", 32, 64, 32, 64, EQUIANGULAR, EQUIANGULAR, 0.3, 1, 1, 16, 0,
                   description="equiangular 32x64, theta=0.3, B=1 H=1 C=16"),
    "c2": Workload("c2", 128, 256, 128, 256, EQUIANGULAR, EQUIANGULAR, 4.0 * math.pi / 127.0, 4, 4, 32, 1,
                   description="equiangular 128x256, theta=4pi/127, B=4 H=4 C=32"),
    "c3": Workload("c3", 256, 512, 128, 256, EQUIANGULAR, EQUIANGULAR, 3.0 * math.pi / 127.0, 2, 8, 32, 2,
                   description="equiangular 256x512 -> 128x256, theta=3pi/127, B=2 H=8 C=32 (headline)"),
    "c4": Workload("c4", 361, 720, 361, 720, LEGENDRE_GAUSS, LEGENDRE_GAUSS, 5.0 * math.pi / 360.0, 1, 8, 32, 3,
                   dout_std=0.1, description="Gauss-Legendre 361x720, theta=5pi/360, B=1 H=8 C=32"),
    "c5": Workload("c5", 64, 128, 64, 128, EQUIANGULAR, EQUIANGULAR, math.pi, 2, 4, 32, 4,
                   description="equiangular 64x128, theta=pi (global limit), B=2 H=4 C=32"),
}


def make_inputs(wl: Workload):
    """float32 host arrays (q, k, v, dout), i.i.d. N(0,1) (dout scaled by dout_std), PCG64(seed)."""
    rng = np.random.Generator(np.random.PCG64(wl.seed))
    q = rng.standard_normal(wl.q_shape, dtype=np.float64).astype(np.float32)
    k = rng.standard_normal(wl.k_shape, dtype=np.float64).astype(np.float32)
    v = rng.standard_normal(wl.k_shape, dtype=np.float64).astype(np.float32)
    dout = (wl.dout_std * rng.standard_normal(wl.q_shape, dtype=np.float64)).astype(np.float32)
    return q, k, v, dout


def small_workload(name, nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, theta_cutoff, B, H, C, seed,
                   dout_std=1.0) -> Workload:
    return Workload(name, nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, theta_cutoff, B, H, C, seed,
                    dout_std)


def sample_points(rng: np.random.Generator, N: int, nlat: int, nlon: int, count: int, polar_rows: int = 2):
    """Random (n, h, w) triples that always include rows next to both poles and the equator."""
    pts = np.stack([rng.integers(0, N, count), rng.integers(0, nlat, count), rng.integers(0, nlon, count)], axis=1)
    forced = [0, nlat - 1, nlat // 2] + list(range(1, 1 + polar_rows)) + list(range(nlat - 1 - polar_rows, nlat - 1))
    for i, h in enumerate(forced[:count]):
        pts[i, 1] = h
    return pts.astype(np.int32)
