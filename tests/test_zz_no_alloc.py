"""GPU test of sna_backward_static, the backward entry point for callers that cannot allocate device memory
(hosts that run inside a pre-sized memory arena, real-time loops, plug-ins that only receive buffers).  Its
scratch is a fixed array inside the library, so the test checks, through the C ABI, that it gives what
sna_backward gives, twice in a row (the array is shared between calls and keeps the previous call's
contents), that the gradients also agree with the fp64 oracle, that the amount of free device memory does not
change across the call, and that a problem beyond the array's capacity is refused.

The file name sorts last on purpose: a run that stops at the first failure has then already run every other
test.  The test is self-contained and passes alone in a fresh process as well as after the others.
"""
import math

import numpy as np
import pytest
import torch

from oracle import sna_oracle as orc
from paper_2505_11157_b200 import sna
from paper_2505_11157_b200.synthetic import make_inputs, small_workload

pytestmark = pytest.mark.gpu

BWD_TOL = 1e-4


def _nerr(x, ref):
    x, ref = x.double(), ref.double()
    return float((x - ref).abs().max() / ref.abs().max())


def test_static_scratch_backward_matches_sna_backward_twice():
    cases = [small_workload("na_down2", 33, 64, 17, 32, 0, 0, 2 * math.pi / 16, 2, 2, 32, 40),
             small_workload("na_gl", 20, 40, 20, 40, 1, 1, 0.5, 1, 3, 16, 41)]
    for call, wl in enumerate(cases):            # two calls in a row, different sizes, same static array
        q, k, v, dout = (torch.from_numpy(a).cuda() for a in make_inputs(wl))
        with sna.Plan(wl.nlat_in, wl.nlon_in, wl.nlat_out, wl.nlon_out, wl.grid_in, wl.grid_out, wl.theta_cutoff) as plan:
            ref = [torch.empty_like(q), torch.empty_like(k), torch.empty_like(k)]
            sna.sna_backward(plan.handle, q, k, v, dout, *ref, wl.B, wl.H, wl.C)
            got = [torch.full_like(q, float("nan")), torch.full_like(k, float("nan")), torch.full_like(k, float("nan"))]
            sna.sna_backward_static(plan.handle, q, k, v, dout, *got, wl.B, wl.H, wl.C)
            torch.cuda.synchronize()
            for name, g, r in zip(("dq", "dk", "dv"), got, ref):
                assert torch.isfinite(g).all(), (call, name)
                assert _nerr(g, r) <= BWD_TOL, (call, name)
            # same inputs again: the array now holds this problem's old statistics
            again = [torch.empty_like(q), torch.empty_like(k), torch.empty_like(k)]
            sna.sna_backward_static(plan.handle, q, k, v, dout, *again, wl.B, wl.H, wl.C)
            torch.cuda.synchronize()
            for name, g, r in zip(("dq", "dk", "dv"), again, ref):
                assert _nerr(g, r) <= BWD_TOL, (call, "repeat", name)


def test_static_scratch_backward_matches_the_oracle_and_allocates_nothing():
    wl = small_workload("na_oracle", 24, 48, 24, 48, 0, 0, 0.45, 1, 3, 32, 42)
    g = orc.geometry(wl.nlat_in, wl.nlon_in, wl.nlat_out, wl.nlon_out, wl.grid_in, wl.grid_out, wl.theta_cutoff)
    hq, hk, hv, hdout = make_inputs(wl)
    q, k, v, dout = (torch.from_numpy(a).cuda() for a in (hq, hk, hv, hdout))
    with sna.Plan(wl.nlat_in, wl.nlon_in, wl.nlat_out, wl.nlon_out, wl.grid_in, wl.grid_out, wl.theta_cutoff) as plan:
        got = [torch.empty_like(q), torch.empty_like(k), torch.empty_like(k)]
        # first call: looks up the array's address on this device (no allocation either, but keep it out of the
        # measured window together with any lazy initialisation of the CUDA context)
        sna.sna_backward_static(plan.handle, q, k, v, dout, *got, wl.B, wl.H, wl.C)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        sna.sna_backward_static(plan.handle, q, k, v, dout, *got, wl.B, wl.H, wl.C)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before, "sna_backward_static changed the amount of free device memory"
    refs = orc.backward(g, hq, hk, hv, hdout)
    for name, x, r in zip(("dq", "dk", "dv"), got, refs):
        x = x.cpu().numpy().astype(np.float64).reshape(r.shape)
        assert np.max(np.abs(x - r)) / np.max(np.abs(r)) <= BWD_TOL, name


def test_static_scratch_rejects_problems_beyond_its_capacity():
    # 1 x 5 x 512 x 512 output points > 2^20: refused on the host before anything is launched
    with sna.Plan(512, 512, 512, 512, 0, 0, 0.02) as plan:
        dummy = torch.zeros(16, device="cuda")
        with pytest.raises(sna.SnaError) as e:
            sna.sna_backward_static(plan.handle, dummy, dummy, dummy, dummy, dummy, dummy, dummy, 1, 5, 32)
        assert e.value.status == sna.SNA_ERR_WORKSPACE
        assert "static scratch" in str(e.value)
    torch.cuda.synchronize()
