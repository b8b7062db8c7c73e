"""Thin Python binding of the C ABI in ``include/sna.h`` (ctypes).

Only argument marshalling happens here: tensors are handed over as raw device pointers, the stream as a
``cudaStream_t``.  Every step of the computation runs in the library's CUDA kernels.  PyTorch provides device
memory and streams, nothing else.  There is no CPU fallback: if the shared library is missing, importing this
module raises.

The module-level functions carry the names of the C entry points; :class:`Plan` is a convenience wrapper
around them.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libsna.so")

SNA_GRID_EQUIANGULAR = 0
SNA_GRID_LEGENDRE_GAUSS = 1
SNA_GRID_EQUIANGULAR_TRAPEZOID = 2

SNA_OK = 0
SNA_ERR_INVALID_ARG = 1
SNA_ERR_UNSUPPORTED = 2
SNA_ERR_EMPTY_NEIGHBORHOOD = 3
SNA_ERR_ALLOC = 4
SNA_ERR_CUDA = 5
SNA_ERR_AMBIGUOUS_TIE = 6
SNA_ERR_WORKSPACE = 7

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it first (python -m paper_2505_11157_b200.build). "
        "There is no fallback implementation.")

_lib = ctypes.CDLL(LIB_PATH)

_vp, _i, _d, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_double, ctypes.c_size_t
_SIGNATURES = {
    "sna_plan_create": (_i, [_i, _i, _i, _i, _i, _i, _d, ctypes.POINTER(_vp)]),
    "sna_plan_create_host_only": (_i, [_i, _i, _i, _i, _i, _i, _d, ctypes.POINTER(_vp)]),
    "sna_debug_exercise_bounded_wait": (_i, [_vp, _i, _vp]),
    "sna_plan_create_global": (_i, [_i, _i, _i, _i, _i, _i, ctypes.POINTER(_vp)]),
    "sna_plan_destroy": (_i, [_vp]),
    "sna_plan_check": (_i, [_vp]),
    "sna_plan_get_nnz": (_i, [_vp, ctypes.POINTER(ctypes.c_int64)]),
    "sna_plan_get_colatitudes": (_i, [_vp, _vp, _vp]),
    "sna_plan_get_quad_weights": (_i, [_vp, _vp]),
    "sna_plan_get_table": (_i, [_vp, _vp, _vp, _vp]),
    "sna_plan_get_table_transposed": (_i, [_vp, _vp, _vp, _vp]),
    "sna_workspace_bytes": (_sz, [_vp, _i, _i, _i]),
    "sna_forward_kernel_count": (_i, [_vp, _i, _i]),
    "sna_forward": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _vp]),
    "sna_forward_ex": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _vp]),
    "sna_backward": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _vp]),
    "sna_backward_ex": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _i, _i, _i, _vp]),
    "sna_backward_dq": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _vp]),
    "sna_backward_dkdv": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _vp]),
    "sna_cf_state_bytes": (_sz, [_vp, _i, _i, _i]),
    "sna_cf_scratch_bytes": (_sz, [_vp, _i, _i, _i]),
    "sna_forward_cf": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _sz, _i, _i, _i, _vp]),
    "sna_backward_cf": (_i, [_vp, _vp, _vp, _sz, _vp, _sz, _vp, _vp, _vp, _i, _i, _i, _vp]),
    "sna_forward_tf32": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _vp]),
    "sna_backward_tf32": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _i, _i, _i, _vp]),
    "sna_backward_static": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _vp]),
    "sna_measure_fp32_fma_peak": (_i, [ctypes.POINTER(ctypes.c_double)]),
    "sna_status_string": (ctypes.c_char_p, [_i]),
    "sna_last_error_message": (ctypes.c_char_p, []),
}
for _name, (_res, _args) in _SIGNATURES.items():
    _fn = getattr(_lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


class SnaError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        name = _lib.sna_status_string(status).decode()
        detail = _lib.sna_last_error_message().decode()
        super().__init__(f"{name}: {detail}" if detail else name)


def _check(status: int):
    if status != SNA_OK:
        raise SnaError(status)


def _ptr(t) -> Optional[int]:
    """Device pointer of a CUDA tensor (or pass through an int / None)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


# ---- functions with the names of the C entry points --------------------------------------------------------

def sna_plan_create(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, theta_cutoff, host_only=False) -> int:
    handle = _vp()
    fn = _lib.sna_plan_create_host_only if host_only else _lib.sna_plan_create
    _check(fn(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, float(theta_cutoff), ctypes.byref(handle)))
    return handle.value


def sna_plan_create_global(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out) -> int:
    """Plan for global spherical attention (every output point attends to every input point)."""
    handle = _vp()
    _check(_lib.sna_plan_create_global(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, ctypes.byref(handle)))
    return handle.value


def sna_debug_exercise_bounded_wait(plan: int, polls: int = 1000, stream=None) -> None:
    """Test aid: make one bounded wait run out on the GPU so that ``sna_plan_check`` has a failure to report."""
    _check(_lib.sna_debug_exercise_bounded_wait(plan, polls, _stream(stream)))


def sna_plan_create_host_only(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, theta_cutoff) -> int:
    return sna_plan_create(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, theta_cutoff, host_only=True)


def sna_plan_destroy(plan: int):
    _check(_lib.sna_plan_destroy(plan))


def sna_plan_check(plan: int):
    """Synchronise and raise if a kernel of this plan gave up on a bounded wait."""
    _check(_lib.sna_plan_check(plan))


def sna_plan_get_nnz(plan: int) -> int:
    n = ctypes.c_int64()
    _check(_lib.sna_plan_get_nnz(plan, ctypes.byref(n)))
    return n.value


def sna_workspace_bytes(plan: int, B: int, H: int, C: int) -> int:
    return int(_lib.sna_workspace_bytes(plan, B, H, C))


def sna_forward_kernel_count(plan: int, C: int, with_lse: bool) -> int:
    return int(_lib.sna_forward_kernel_count(plan, C, 1 if with_lse else 0))


def sna_forward(plan, q, k, v, out, B, H, C, stream=None):
    _check(_lib.sna_forward(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, C, _stream(stream)))


def sna_forward_ex(plan, q, k, v, out, lse, B, H, C, stream=None):
    _check(_lib.sna_forward_ex(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), B, H, C, _stream(stream)))


def sna_backward(plan, q, k, v, dout, dq, dk, dv, B, H, C, stream=None):
    _check(_lib.sna_backward(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(dq), _ptr(dk), _ptr(dv), B, H, C,
                             _stream(stream)))


def sna_backward_ex(plan, q, k, v, dout, out, lse, dq, dk, dv, workspace, workspace_bytes, B, H, C, stream=None):
    _check(_lib.sna_backward_ex(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(out), _ptr(lse), _ptr(dq), _ptr(dk),
                                _ptr(dv), _ptr(workspace), workspace_bytes, B, H, C, _stream(stream)))


def sna_backward_dq(plan, q, k, v, dout, out, lse, dq, D, B, H, C, stream=None):
    _check(_lib.sna_backward_dq(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(out), _ptr(lse), _ptr(dq), _ptr(D),
                                B, H, C, _stream(stream)))


def sna_backward_dkdv(plan, q, k, v, dout, lse, D, dk, dv, B, H, C, stream=None):
    _check(_lib.sna_backward_dkdv(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(lse), _ptr(D), _ptr(dk), _ptr(dv),
                                  B, H, C, _stream(stream)))


def sna_forward_tf32(plan, q, k, v, out, lse, B, H, C, stream=None):
    """Reduced-precision forward pass (one TF32 product per contraction; normalised error below 5e-3)."""
    _check(_lib.sna_forward_tf32(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), B, H, C, _stream(stream)))


def sna_backward_tf32(plan, q, k, v, dout, out, lse, dq, dk, dv, workspace, workspace_bytes, B, H, C, stream=None):
    """Reduced-precision backward pass; arguments as sna_backward_ex."""
    _check(_lib.sna_backward_tf32(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(out), _ptr(lse), _ptr(dq), _ptr(dk),
                                  _ptr(dv), _ptr(workspace), workspace_bytes, B, H, C, _stream(stream)))


SNA_STATIC_SCRATCH_MAX_POINTS = 1 << 20


def sna_backward_static(plan, q, k, v, dout, dq, dk, dv, B, H, C, stream=None):
    """Backward pass that allocates nothing: its scratch is a fixed array inside the library (at most
    SNA_STATIC_SCRATCH_MAX_POINTS output points).  For callers that cannot call cudaMalloc; calls whose GPU work
    overlaps share that array and must be serialised."""
    _check(_lib.sna_backward_static(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(dq), _ptr(dk), _ptr(dv),
                                    B, H, C, _stream(stream)))


def sna_measure_fp32_fma_peak() -> float:
    """Sustained FP32 FMA rate of the current device in TFLOP/s (a pure-FMA loop on every SM)."""
    t = ctypes.c_double()
    _check(_lib.sna_measure_fp32_fma_peak(ctypes.byref(t)))
    return t.value


# ---- convenience wrapper -----------------------------------------------------------------------------------

def sna_cf_state_bytes(plan: int, B: int, H: int, C: int) -> int:
    return int(_lib.sna_cf_state_bytes(plan, B, H, C))


def sna_cf_scratch_bytes(plan: int, B: int, H: int, C: int) -> int:
    return int(_lib.sna_cf_scratch_bytes(plan, B, H, C))


def sna_forward_cf(plan, q_cf, k_cf, v_cf, out_cf, state, state_bytes, B, H, C, stream=None) -> None:
    _check(_lib.sna_forward_cf(plan, _ptr(q_cf), _ptr(k_cf), _ptr(v_cf), _ptr(out_cf), _ptr(state), state_bytes, B, H, C,
                               _stream(stream)))


def sna_backward_cf(plan, dout_cf, state, state_bytes, scratch, scratch_bytes, dq_cf, dk_cf, dv_cf, B, H, C, stream=None) -> None:
    _check(_lib.sna_backward_cf(plan, _ptr(dout_cf), _ptr(state), state_bytes, _ptr(scratch), scratch_bytes,
                                _ptr(dq_cf), _ptr(dk_cf), _ptr(dv_cf), B, H, C, _stream(stream)))


class Plan:
    """Owns one ``sna_plan_t``.  Shapes follow the header: q/out [B,H,nlat_out,nlon_out,C], k/v [B,H,nlat_in,nlon_in,C]."""

    def __init__(self, nlat_in, nlon_in, nlat_out, nlon_out, grid_in=SNA_GRID_EQUIANGULAR,
                 grid_out=SNA_GRID_EQUIANGULAR, theta_cutoff=0.1, host_only=False, global_attention=False):
        self.nlat_in, self.nlon_in, self.nlat_out, self.nlon_out = nlat_in, nlon_in, nlat_out, nlon_out
        self.grid_in, self.grid_out, self.theta_cutoff = grid_in, grid_out, float(theta_cutoff)
        self.host_only = host_only
        self.handle = None
        if global_attention:
            self.handle = sna_plan_create_global(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out)
        else:
            self.handle = sna_plan_create(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, theta_cutoff, host_only)
        self.ps = nlon_in // nlon_out

    def close(self):
        if self.handle is not None:
            handle, self.handle = self.handle, None
            sna_plan_destroy(handle)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # introspection (host)
    @property
    def nnz(self) -> int:
        return sna_plan_get_nnz(self.handle)

    def colatitudes(self):
        ti = np.empty(self.nlat_in, dtype=np.float64)
        to = np.empty(self.nlat_out, dtype=np.float64)
        _check(_lib.sna_plan_get_colatitudes(self.handle, ti.ctypes.data, to.ctypes.data))
        return ti, to

    def quad_weights(self):
        w = np.empty(self.nlat_in, dtype=np.float64)
        _check(_lib.sna_plan_get_quad_weights(self.handle, w.ctypes.data))
        return w

    def table(self):
        nnz = self.nnz
        row_ptr = np.empty(self.nlat_out + 1, dtype=np.int64)
        lat = np.empty(nnz, dtype=np.int32)
        off = np.empty(nnz, dtype=np.int32)
        _check(_lib.sna_plan_get_table(self.handle, row_ptr.ctypes.data, lat.ctypes.data, off.ctypes.data))
        return row_ptr, lat, off

    def table_transposed(self):
        nnz = self.nnz
        row_ptr = np.empty(self.nlat_in * self.ps + 1, dtype=np.int64)
        lat = np.empty(nnz, dtype=np.int32)
        off = np.empty(nnz, dtype=np.int32)
        _check(_lib.sna_plan_get_table_transposed(self.handle, row_ptr.ctypes.data, lat.ctypes.data, off.ctypes.data))
        return row_ptr, lat, off

    # compute (device tensors)
    def _bhc(self, q, k):
        if q.dim() != 5 or k.dim() != 5:
            raise ValueError("q and k must be [B, H, nlat, nlon, C]")
        B, H, C = q.shape[0], q.shape[1], q.shape[4]
        if tuple(q.shape[2:4]) != (self.nlat_out, self.nlon_out) or tuple(k.shape) != (B, H, self.nlat_in, self.nlon_in, C):
            raise ValueError("tensor shapes do not match the plan")
        return B, H, C

    def _validate(self, q, **tensors):
        """The kernels read raw pointers as contiguous fp32 of the plan's shapes: refuse anything else here, on the
        host, instead of letting a kernel run past an allocation.  Keyword names select the expected shape:
        out-grid tensors (q, out, dout, dq), in-grid tensors (k, v, dk, dv) and per-point statistics (lse)."""
        import torch
        B, H, C = q.shape[0], q.shape[1], q.shape[4]
        out_shape = (B, H, self.nlat_out, self.nlon_out, C)
        in_shape = (B, H, self.nlat_in, self.nlon_in, C)
        expected = {"q": out_shape, "out": out_shape, "dout": out_shape, "dq": out_shape,
                    "k": in_shape, "v": in_shape, "dk": in_shape, "dv": in_shape, "lse": out_shape[:-1]}
        given = {name: t for name, t in dict(q=q, **tensors).items() if t is not None}
        for name, t in given.items():
            if not isinstance(t, torch.Tensor):
                raise ValueError(f"{name} must be a torch.Tensor")
            if t.dtype != torch.float32:
                raise ValueError(f"{name} must be float32, got {t.dtype}")
            if tuple(t.shape) != expected[name]:
                raise ValueError(f"{name} has shape {tuple(t.shape)}, expected {expected[name]}")
            if not t.is_contiguous():
                raise ValueError(f"{name} must be contiguous")
        for name, t in given.items():
            if not t.is_cuda or t.device != q.device:
                raise ValueError(f"{name} must be a CUDA tensor on the device of q ({q.device}), got {t.device}")

    def workspace_bytes(self, B, H, C) -> int:
        return sna_workspace_bytes(self.handle, B, H, C)

    def forward(self, q, k, v, out=None, lse=None, return_lse=False, stream=None, precision="fp32"):
        """precision: "fp32" (default, error-compensated products) or "tf32" (reduced-precision variant)."""
        import torch
        B, H, C = self._bhc(q, k)
        self._validate(q, k=k, v=v, out=out, lse=lse)
        if precision not in ("fp32", "tf32"):
            raise ValueError("precision must be 'fp32' or 'tf32'")
        if out is None:
            out = torch.empty_like(q)
        if return_lse and lse is None:
            lse = torch.empty(q.shape[:-1], dtype=torch.float32, device=q.device)
        (sna_forward_ex if precision == "fp32" else sna_forward_tf32)(self.handle, q, k, v, out, lse, B, H, C, stream)
        return (out, lse) if return_lse else out

    def _validate_cf(self, heads, **tensors):
        """Channels-first tensors [B, heads*C, nlat, nlon]: out-grid (q, out, dout, dq) or in-grid (k, v, dk, dv)."""
        import torch
        q = tensors["q"] if "q" in tensors else tensors["dout"]
        if not isinstance(q, torch.Tensor) or q.dim() != 4 or heads < 1 or q.shape[1] % heads != 0:
            raise ValueError("channels-first tensors must be [B, heads*C, nlat, nlon]")
        B, HC = q.shape[0], q.shape[1]
        out_shape, in_shape = (B, HC, self.nlat_out, self.nlon_out), (B, HC, self.nlat_in, self.nlon_in)
        expected = {"q": out_shape, "out": out_shape, "dout": out_shape, "dq": out_shape,
                    "k": in_shape, "v": in_shape, "dk": in_shape, "dv": in_shape}
        for name, t in tensors.items():
            if t is None:
                continue
            if not isinstance(t, torch.Tensor) or t.dtype != torch.float32:
                raise ValueError(f"{name} must be a float32 torch.Tensor")
            if tuple(t.shape) != expected[name]:
                raise ValueError(f"{name} has shape {tuple(t.shape)}, expected {expected[name]}")
            if not t.is_contiguous():
                raise ValueError(f"{name} must be contiguous")
            if not t.is_cuda or t.device != q.device:
                raise ValueError(f"{name} must be a CUDA tensor on the device of the first tensor ({q.device})")
        return B, heads, HC // heads

    def forward_cf(self, q, k, v, heads, out=None, state=None, stream=None):
        """Channels-first forward: q [B, heads*C, nlat_out, nlon_out], k, v [B, heads*C, nlat_in, nlon_in].
        Returns (out, state); pass the state to backward_cf."""
        import torch
        B, H, C = self._validate_cf(heads, q=q, k=k, v=v, out=out)
        need = sna_cf_state_bytes(self.handle, B, H, C)
        if state is None:
            state = torch.empty(need, dtype=torch.uint8, device=q.device)
        elif not state.is_cuda or state.device != q.device or not state.is_contiguous():
            raise ValueError("state must be a contiguous CUDA tensor on the device of q")
        out = torch.empty_like(q) if out is None else out
        sna_forward_cf(self.handle, q, k, v, out, state, state.numel() * state.element_size(), B, H, C, stream)
        return out, state

    def backward_cf(self, dout, state, heads, dq=None, dk=None, dv=None, scratch=None, stream=None):
        """Channels-first backward from the state forward_cf left: returns (dq, dk, dv), channels first."""
        import torch
        B, H, C = self._validate_cf(heads, dout=dout, dq=dq, dk=dk, dv=dv)
        need = sna_cf_scratch_bytes(self.handle, B, H, C)
        if scratch is None:
            scratch = torch.empty(need, dtype=torch.uint8, device=dout.device)
        for name, t in (("state", state), ("scratch", scratch)):
            if not isinstance(t, torch.Tensor) or not t.is_cuda or t.device != dout.device or not t.is_contiguous():
                raise ValueError(f"{name} must be a contiguous CUDA tensor on the device of dout")
        in_shape = (B, H * C, self.nlat_in, self.nlon_in)
        dq = torch.empty_like(dout) if dq is None else dq
        dk = torch.empty(in_shape, dtype=torch.float32, device=dout.device) if dk is None else dk
        dv = torch.empty(in_shape, dtype=torch.float32, device=dout.device) if dv is None else dv
        sna_backward_cf(self.handle, dout, state, state.numel() * state.element_size(), scratch,
                        scratch.numel() * scratch.element_size(), dq, dk, dv, B, H, C, stream)
        return dq, dk, dv

    def backward(self, q, k, v, dout, out=None, lse=None, dq=None, dk=None, dv=None, workspace=None, stream=None,
                 precision="fp32"):
        import torch
        B, H, C = self._bhc(q, k)
        if precision not in ("fp32", "tf32"):
            raise ValueError("precision must be 'fp32' or 'tf32'")
        self._validate(q, k=k, v=v, dout=dout, out=out, lse=lse, dq=dq, dk=dk, dv=dv)
        if workspace is not None and (not workspace.is_cuda or workspace.device != q.device or not workspace.is_contiguous()):
            raise ValueError("workspace must be a contiguous CUDA tensor on the device of q")
        dq = torch.empty_like(q) if dq is None else dq
        dk = torch.empty_like(k) if dk is None else dk
        dv = torch.empty_like(k) if dv is None else dv
        if precision == "tf32":
            need = self.workspace_bytes(B, H, C)
            if workspace is None:
                workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
            sna_backward_tf32(self.handle, q, k, v, dout, out, lse, dq, dk, dv, workspace,
                              workspace.numel() * workspace.element_size(), B, H, C, stream)
        elif workspace is None and out is None and lse is None:
            sna_backward(self.handle, q, k, v, dout, dq, dk, dv, B, H, C, stream)
        else:
            need = self.workspace_bytes(B, H, C)
            if workspace is None:
                workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
            sna_backward_ex(self.handle, q, k, v, dout, out, lse, dq, dk, dv, workspace, workspace.numel() * workspace.element_size(), B, H, C, stream)
        return dq, dk, dv
