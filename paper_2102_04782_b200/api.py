"""Thin Python binding of libdai8.so (ctypes).  Same names as ``include/dai8.h``.

Argument marshalling only: tensors are torch CUDA tensors used as device buffers, every step of
the path runs in the library's kernels.  The shared library must have been built
(``python -m paper_2102_04782_b200.build``); a missing library is an error, there is no fallback.
"""
from __future__ import annotations

import ctypes
from ctypes import c_int, c_size_t, c_uint32, c_uint64, c_void_p
from pathlib import Path
from typing import Optional

import torch

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA, ERR_TIMEOUT = range(7)
F32, BF16, I32 = 0, 1, 2
NCHW, NHWC = 0, 1
ROUND_NEAREST_EVEN, ROUND_STOCHASTIC = 0, 1
SCALE_ABSMAX, SCALE_GIVEN = 0, 1
OP_FWD, OP_BWD_DATA, OP_BWD_FILTER = 0, 1, 2
GRAD_FULL, GRAD_GQ, GRAD_GVQ_MAX, GRAD_LAYER_MCS = 0, 1, 2, 3

EXPORTS = [
    "dai8_status_string", "dai8_mcs_defaults", "dai8_padded_channels", "dai8_quantize_tensor",
    "dai8_quantize_tensor_workspace_bytes",
    "dai8_quantize_grad_workspace_bytes", "dai8_quantize_grad", "dai8_quantize_grad_noalloc",
    "dai8_conv_workspace_bytes",
    "dai8_conv_fwd", "dai8_conv_bwd_data", "dai8_conv_bwd_filter", "dai8_set_conv_backend",
    "dai8_launch_count", "dai8_get_device_status", "dai8_debug_expire_waits",
    "dai8_debug_probe_mma", "dai8_debug_probe_sr",
    "dai8_conv3d_fwd", "dai8_conv3d_bwd_data", "dai8_conv3d_bwd_filter",
    "dai8_debug_last_kernel",
    "dai8_dp_grad_workspace_bytes", "dai8_dp_grad_pivot", "dai8_dp_grad_moments", "dai8_dp_grad_sigma", "dai8_dp_grad_count",
    "dai8_dp_grad_solve", "dai8_dp_grad_codes", "dai8_absmax", "dai8_dequant_filter",
]


class ConvGeom(ctypes.Structure):
    _fields_ = [(n, c_int) for n in ("N", "Cin", "Cout", "H", "W", "R", "S", "stride_h", "stride_w",
                                     "pad_h", "pad_w")]

    @property
    def P(self) -> int:
        return (self.H + 2 * self.pad_h - self.R) // self.stride_h + 1

    @property
    def Q(self) -> int:
        return (self.W + 2 * self.pad_w - self.S) // self.stride_w + 1


class Conv3dGeom(ctypes.Structure):
    _fields_ = [(n, c_int) for n in ("N", "Cin", "Cout", "D", "H", "W", "T", "R", "S", "stride_d", "stride_h",
                                     "stride_w", "pad_d", "pad_h", "pad_w", "groups")]

    def out_dhw(self):
        return ((self.D + 2 * self.pad_d - self.T) // self.stride_d + 1,
                (self.H + 2 * self.pad_h - self.R) // self.stride_h + 1,
                (self.W + 2 * self.pad_w - self.S) // self.stride_w + 1)


class McsParams(ctypes.Structure):
    _fields_ = [("lam", ctypes.c_float), ("k", ctypes.c_float), ("A", ctypes.c_float),
                ("std_unbiased", c_int), ("center_mean", c_int), ("mode", c_int)]


class Dai8Error(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


_LIB_PATH = Path(__file__).resolve().parent / "libdai8.so"
_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with "
                               "`python -m paper_2102_04782_b200.build` (there is no CPU fallback)")
        l = ctypes.CDLL(str(_LIB_PATH))
        l.dai8_status_string.restype = ctypes.c_char_p
        l.dai8_status_string.argtypes = [c_int]
        l.dai8_mcs_defaults.restype = None
        l.dai8_padded_channels.restype = c_int
        l.dai8_quantize_grad_workspace_bytes.restype = c_size_t
        l.dai8_quantize_grad_workspace_bytes.argtypes = [c_int]
        l.dai8_conv_workspace_bytes.restype = c_size_t
        l.dai8_conv_workspace_bytes.argtypes = [c_int, ctypes.POINTER(ConvGeom)]
        l.dai8_launch_count.restype = c_uint64
        l.dai8_set_conv_backend.restype = None
        l.dai8_quantize_tensor_workspace_bytes.restype = c_size_t
        l.dai8_quantize_tensor_workspace_bytes.argtypes = []
        l.dai8_quantize_tensor.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_int, c_int,
                                           c_void_p, c_int, c_uint32, c_void_p, c_void_p, c_size_t, c_void_p]
        l.dai8_quantize_grad.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_int,
                                         ctypes.POINTER(McsParams), c_void_p, c_int, c_void_p,
                                         c_void_p, c_void_p, c_void_p, c_void_p, c_uint32, c_void_p,
                                         c_void_p, c_size_t, c_void_p]
        l.dai8_quantize_grad_noalloc.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_int,
                                                 ctypes.POINTER(McsParams), c_void_p, c_int, c_void_p,
                                                 c_void_p, c_void_p, c_void_p, c_void_p, c_uint32,
                                                 c_void_p]
        conv_args = [c_void_p, c_void_p, c_void_p, c_void_p, ctypes.POINTER(ConvGeom), c_void_p, c_int,
                     c_int, c_void_p, c_size_t, c_void_p]
        l.dai8_conv_fwd.argtypes = conv_args
        l.dai8_conv_bwd_data.argtypes = conv_args
        l.dai8_conv_bwd_filter.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p,
                                           ctypes.POINTER(ConvGeom), c_void_p, c_int, c_void_p,
                                           c_size_t, c_void_p]
        l.dai8_get_device_status.argtypes = [ctypes.POINTER(c_int), c_void_p]
        c_i64 = ctypes.c_int64
        l.dai8_dp_grad_workspace_bytes.argtypes = [c_int]
        l.dai8_dp_grad_workspace_bytes.restype = ctypes.c_size_t
        l.dai8_dp_grad_pivot.argtypes = [c_void_p, c_int, c_int, c_int, c_void_p, c_void_p]
        l.dai8_dp_grad_moments.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_int, c_void_p, c_void_p,
                                           c_void_p, c_void_p, ctypes.c_size_t, c_void_p]
        l.dai8_dp_grad_sigma.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_i64, ctypes.POINTER(McsParams),
                                         c_void_p, c_void_p, c_void_p, c_void_p]
        l.dai8_dp_grad_count.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_int, c_void_p, c_void_p,
                                         c_void_p, ctypes.c_size_t, c_void_p]
        l.dai8_dp_grad_solve.argtypes = [c_void_p, c_void_p, c_int, c_i64, ctypes.POINTER(McsParams), c_void_p, c_int,
                                         c_void_p, c_void_p]
        l.dai8_dp_grad_codes.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_int, c_i64, c_void_p, c_void_p,
                                         ctypes.c_uint32, c_void_p, c_void_p, c_void_p]
        l.dai8_absmax.argtypes = [c_void_p, c_int, c_i64, c_void_p, c_void_p]
        l.dai8_dequant_filter.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_i64, c_void_p, c_void_p]
        l.dai8_debug_last_kernel.argtypes = []
        l.dai8_debug_last_kernel.restype = ctypes.c_char_p
        nd_args = [c_void_p, c_void_p, c_void_p, c_void_p, ctypes.POINTER(Conv3dGeom), c_void_p, c_int, c_void_p]
        l.dai8_conv3d_fwd.argtypes = nd_args
        l.dai8_conv3d_bwd_data.argtypes = nd_args
        l.dai8_conv3d_bwd_filter.argtypes = nd_args
        l.dai8_debug_expire_waits.argtypes = [c_uint64, ctypes.POINTER(c_int), c_void_p, c_size_t, c_void_p]
        dp = ctypes.POINTER(ctypes.c_double)
        l.dai8_debug_probe_mma.argtypes = [c_int, c_int, c_int, dp, dp, c_void_p, c_size_t, c_void_p]
        l.dai8_debug_probe_sr.argtypes = [c_int, dp, c_void_p, c_size_t, c_void_p]
        _lib = l
    return _lib


def status_string(code: int) -> str:
    return lib().dai8_status_string(code).decode()


def _check(code: int, where: str) -> None:
    if code != OK:
        raise Dai8Error(code, where)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("dai8 takes CUDA tensors (device buffers)")
    if not t.is_contiguous():
        raise ValueError("dai8 takes contiguous buffers")
    return c_void_p(t.data_ptr())


def _stream() -> c_void_p:
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.int32:
        return I32
    raise ValueError(f"unsupported dtype {t.dtype}")


def padded_channels(C: int) -> int:
    return int(lib().dai8_padded_channels(C))


def mcs_defaults() -> McsParams:
    p = McsParams()
    lib().dai8_mcs_defaults(ctypes.byref(p))
    return p


def launch_count() -> int:
    return int(lib().dai8_launch_count())


def set_conv_backend(mode: int) -> None:
    lib().dai8_set_conv_backend(mode)


def get_device_status() -> int:
    v = c_int(0)
    _check(lib().dai8_get_device_status(ctypes.byref(v), _stream()), "dai8_get_device_status")
    return v.value


def debug_expire_waits(limit_cycles: int, ws: torch.Tensor):
    """dai8_debug_expire_waits: runs the bounded-wait helpers on barriers nobody completes; returns the
    three flags (1 = the wait gave up by itself)."""
    rep = (c_int * 3)()
    p, n = _ws_args(ws)
    _check(lib().dai8_debug_expire_waits(limit_cycles, rep, p, n, _stream()), "dai8_debug_expire_waits")
    return list(rep)


def debug_probe_mma(n_cols: int, row_bytes: int, count: int, ws: torch.Tensor):
    """dai8_debug_probe_mma: (issue, complete) cycles per tcgen05.mma.kind::i8 with operands in shared memory."""
    a, b = ctypes.c_double(0), ctypes.c_double(0)
    p, n = _ws_args(ws)
    _check(lib().dai8_debug_probe_mma(n_cols, row_bytes, count, ctypes.byref(a), ctypes.byref(b), p, n, _stream()),
           "dai8_debug_probe_mma")
    return a.value, b.value


def debug_probe_sr(iters: int, ws: torch.Tensor) -> float:
    """dai8_debug_probe_sr: elements per second of the code sweep's arithmetic in registers."""
    v = ctypes.c_double(0)
    p, n = _ws_args(ws)
    _check(lib().dai8_debug_probe_sr(iters, ctypes.byref(v), p, n, _stream()), "dai8_debug_probe_sr")
    return v.value


def quantize_tensor_workspace_bytes() -> int:
    return int(lib().dai8_quantize_tensor_workspace_bytes())


def quantize_tensor(x: torch.Tensor, layout: int, N: int, C: int, H: int, W: int, scale_mode: int,
                    scale: torch.Tensor, rounding: int, seed: int, q: torch.Tensor,
                    ws: Optional[torch.Tensor] = None) -> None:
    """dai8_quantize_tensor: x (fp32/bf16, `layout`) -> q int8 [N][H][W][Cp]; scale: 1 float;
    ws: scratch of quantize_tensor_workspace_bytes() bytes or None."""
    p, n = _ws_args(ws)
    _check(lib().dai8_quantize_tensor(_ptr(x), _dtype_code(x), layout, N, C, H, W, scale_mode,
                                      _ptr(scale), rounding, seed & 0xFFFFFFFF, _ptr(q), p, n, _stream()),
           "dai8_quantize_tensor")


def quantize_grad_workspace_bytes(C: int) -> int:
    return int(lib().dai8_quantize_grad_workspace_bytes(C))


def quantize_grad(dY: torch.Tensor, layout: int, N: int, C: int, H: int, W: int,
                  params: Optional[McsParams], s_state: torch.Tensor, has_prev: bool,
                  gmax_layer: torch.Tensor, stats: Optional[torch.Tensor],
                  cls: Optional[torch.Tensor], vq: torch.Tensor, gq: Optional[torch.Tensor],
                  seed: int, ws: torch.Tensor, sigma_override: Optional[torch.Tensor] = None) -> None:
    """dai8_quantize_grad (Algorithm 1 up to and including the two quantizations of dY)."""
    _check(lib().dai8_quantize_grad(_ptr(dY), _dtype_code(dY), layout, N, C, H, W,
                                    ctypes.byref(params) if params is not None else None,
                                    _ptr(s_state), int(has_prev), _ptr(gmax_layer), _ptr(stats),
                                    _ptr(cls), _ptr(vq), _ptr(gq), seed & 0xFFFFFFFF,
                                    _ptr(sigma_override), _ptr(ws), ws.numel() * ws.element_size(),
                                    _stream()), "dai8_quantize_grad")


NOALLOC_MAX_CHANNELS = 256


def quantize_grad_noalloc(dY: torch.Tensor, layout: int, N: int, C: int, H: int, W: int,
                          params: Optional[McsParams], s_state: torch.Tensor, has_prev: bool,
                          gmax_layer: torch.Tensor, stats: Optional[torch.Tensor],
                          cls: Optional[torch.Tensor], vq: torch.Tensor,
                          gq: Optional[torch.Tensor], seed: int) -> None:
    """dai8_quantize_grad_noalloc: dai8_quantize_grad for a caller that has no scratch buffer to
    give (it cannot allocate device memory where it runs).  The scratch is a fixed 3 MiB array
    inside the library, shared by all calls on the device, so calls must not overlap on the GPU;
    C is limited to NOALLOC_MAX_CHANNELS."""
    _check(lib().dai8_quantize_grad_noalloc(_ptr(dY), _dtype_code(dY), layout, N, C, H, W,
                                            ctypes.byref(params) if params is not None else None,
                                            _ptr(s_state), int(has_prev), _ptr(gmax_layer),
                                            _ptr(stats), _ptr(cls), _ptr(vq), _ptr(gq),
                                            seed & 0xFFFFFFFF, _stream()),
           "dai8_quantize_grad_noalloc")


def conv_workspace_bytes(op: int, geom: ConvGeom) -> int:
    return int(lib().dai8_conv_workspace_bytes(op, ctypes.byref(geom)))


def _ws_args(ws: Optional[torch.Tensor]):
    if ws is None:
        return None, 0
    return _ptr(ws), ws.numel() * ws.element_size()


def conv_fwd(qX, qW, sX, sW, geom: ConvGeom, Y: torch.Tensor, out_layout: int, ws=None) -> None:
    p, n = _ws_args(ws)
    _check(lib().dai8_conv_fwd(_ptr(qX), _ptr(qW), _ptr(sX), _ptr(sW), ctypes.byref(geom), _ptr(Y),
                               _dtype_code(Y), out_layout, p, n, _stream()), "dai8_conv_fwd")


def conv_bwd_data(gq, qW, gmax, sW, geom: ConvGeom, dX: torch.Tensor, out_layout: int, ws) -> None:
    p, n = _ws_args(ws)
    _check(lib().dai8_conv_bwd_data(_ptr(gq), _ptr(qW), _ptr(gmax), _ptr(sW), ctypes.byref(geom),
                                    _ptr(dX), _dtype_code(dX), out_layout, p, n, _stream()),
           "dai8_conv_bwd_data")


def conv_bwd_filter(qX, vq, sX, s, geom: ConvGeom, dW: torch.Tensor, ws) -> None:
    p, n = _ws_args(ws)
    _check(lib().dai8_conv_bwd_filter(_ptr(qX), _ptr(vq), _ptr(sX), _ptr(s), ctypes.byref(geom),
                                      _ptr(dW), _dtype_code(dW), p, n, _stream()),
           "dai8_conv_bwd_filter")


def conv3d_fwd(qX, qW, sX, sW, geom: Conv3dGeom, Y: torch.Tensor) -> None:
    """dai8_conv3d_fwd: codes [N][D][H][W][Cp] x [Cout][T][R][S][Cgp] -> Y [N][Do][P][Q][Cout]."""
    _check(lib().dai8_conv3d_fwd(_ptr(qX), _ptr(qW), _ptr(sX), _ptr(sW), ctypes.byref(geom), _ptr(Y), _dtype_code(Y),
                                 _stream()), "dai8_conv3d_fwd")


def conv3d_bwd_data(gq, qW, gmax, sW, geom: Conv3dGeom, dX: torch.Tensor) -> None:
    _check(lib().dai8_conv3d_bwd_data(_ptr(gq), _ptr(qW), _ptr(gmax), _ptr(sW), ctypes.byref(geom), _ptr(dX),
                                      _dtype_code(dX), _stream()), "dai8_conv3d_bwd_data")


def conv3d_bwd_filter(qX, vq, sX, s, geom: Conv3dGeom, dW: torch.Tensor) -> None:
    _check(lib().dai8_conv3d_bwd_filter(_ptr(qX), _ptr(vq), _ptr(sX), _ptr(s), ctypes.byref(geom), _ptr(dW),
                                        _dtype_code(dW), _stream()), "dai8_conv3d_bwd_filter")


def debug_last_kernel() -> str:
    """Name of the kernel family the calling thread's last library call launched."""
    return lib().dai8_debug_last_kernel().decode()


# ---- batch-sharded (data-parallel) stages ---------------------------------------------------------
def dp_grad_workspace_bytes(C: int) -> int:
    return int(lib().dai8_dp_grad_workspace_bytes(C))


def _pp(params):
    return ctypes.byref(params) if params is not None else None


def dp_grad_pivot(dY, layout, C, pivot) -> None:
    _check(lib().dai8_dp_grad_pivot(_ptr(dY), _dtype_code(dY), layout, C, _ptr(pivot), _stream()), "dai8_dp_grad_pivot")


def dp_grad_moments(dY, layout, N_local, C, H, W, pivot, absmax, sums, ws) -> None:
    _check(lib().dai8_dp_grad_moments(_ptr(dY), _dtype_code(dY), layout, N_local, C, H, W, _ptr(pivot), _ptr(absmax),
                                      _ptr(sums), _ptr(ws), ws.numel() * ws.element_size(), _stream()),
           "dai8_dp_grad_moments")


def dp_grad_sigma(absmax, sums, pivot, C, M_global, params, mean, sigma, gmax_layer) -> None:
    _check(lib().dai8_dp_grad_sigma(_ptr(absmax), _ptr(sums), _ptr(pivot), C, M_global, _pp(params), _ptr(mean),
                                    _ptr(sigma), _ptr(gmax_layer), _stream()), "dai8_dp_grad_sigma")


def dp_grad_count(dY, layout, N_local, C, H, W, sigma, cnt, ws) -> None:
    _check(lib().dai8_dp_grad_count(_ptr(dY), _dtype_code(dY), layout, N_local, C, H, W, _ptr(sigma), _ptr(cnt),
                                    _ptr(ws), ws.numel() * ws.element_size(), _stream()), "dai8_dp_grad_count")


def dp_grad_solve(cnt, absmax, C, M_global, params, s_state, has_prev, cls) -> None:
    _check(lib().dai8_dp_grad_solve(_ptr(cnt), _ptr(absmax), C, M_global, _pp(params), _ptr(s_state), int(has_prev),
                                    _ptr(cls), _stream()), "dai8_dp_grad_solve")


def dp_grad_codes(dY, layout, N_local, C, H, W, first_image, s, gmax_layer, seed, vq, gq) -> None:
    _check(lib().dai8_dp_grad_codes(_ptr(dY), _dtype_code(dY), layout, N_local, C, H, W, first_image, _ptr(s),
                                    _ptr(gmax_layer), seed & 0xFFFFFFFF, _ptr(vq), _ptr(gq), _stream()),
           "dai8_dp_grad_codes")


def absmax(x, out) -> None:
    _check(lib().dai8_absmax(_ptr(x), _dtype_code(x), x.numel(), _ptr(out), _stream()), "dai8_absmax")


def dequant_filter(acc, sX, s, Cout, per_cout, dW) -> None:
    _check(lib().dai8_dequant_filter(_ptr(acc), _ptr(sX), _ptr(s), Cout, per_cout, _ptr(dW), _stream()),
           "dai8_dequant_filter")
