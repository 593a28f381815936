"""ctypes front end of the C++ oracle (``dai8_oracle.cpp``).  Test infrastructure only.

All tensors are numpy arrays in plain NCHW / (Cout,Cin,R,S) order.  Every function returns new
arrays; none of them touches a GPU.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "dai8_oracle.cpp"
_SO = _HERE / "libdai8_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with g++ (no fused multiply-add contraction, OpenMP across channels)."""
    if force or not _SO.exists() or _SO.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _SO.with_suffix(f".tmp{os.getpid()}.so")
        cmd = ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-o", str(tmp), str(_SRC)]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _SO)
    return _SO


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        _lib.dai8o_rand_uniform.restype = ctypes.c_float
        _lib.dai8o_rand_uniform.argtypes = [ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint64]
        _lib.dai8o_rand_bits.restype = ctypes.c_uint32
        _lib.dai8o_rand_bits.argtypes = [ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint64]
        _lib.dai8o_num_threads.restype = ctypes.c_int
        for name in ("dai8o_conv_fwd_acc", "dai8o_conv_bwd_data_acc", "dai8o_conv_bwd_filter_acc", "dai8o_conv3_acc"):
            getattr(_lib, name).restype = ctypes.c_int64
    return _lib


def num_threads() -> int:
    return int(lib().dai8o_num_threads())


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def channel_stats(g, std_unbiased: bool = False, center_mean: bool = True):
    """Algorithm 1, statistics step.  Returns (absmax[C], mean[C], sigma[C], gmax_layer) as fp32."""
    g = _f32(g)
    N, C, H, W = g.shape
    absmax = np.empty(C, np.float32)
    mean = np.empty(C, np.float32)
    sigma = np.empty(C, np.float32)
    gl = np.empty(1, np.float32)
    lib().dai8o_channel_stats(_p(g), N, C, H, W, int(std_unbiased), int(center_mean), _p(absmax),
                              _p(mean), _p(sigma), _p(gl))
    return absmax, mean, sigma, float(gl[0])


def density_count(g, sigma) -> np.ndarray:
    """Algorithm 1, density step: #{|g| > sigma_c} per channel (uint32)."""
    g = _f32(g)
    sigma = _f32(sigma)
    N, C, H, W = g.shape
    assert sigma.shape == (C,)
    cnt = np.empty(C, np.uint32)
    lib().dai8o_density_count(_p(g), N, C, H, W, _p(sigma), _p(cnt))
    return cnt


def classify_clip(cnt, absmax, M: int, s_prev=None, lam: float = 0.3, k: float = 1.0,
                  A: float = 0.8):
    """Algorithm 1, discriminator and clip update.  Returns (s_t[C] fp32, cls[C] uint8 with 1 = bell-shaped)."""
    cnt = np.ascontiguousarray(cnt, dtype=np.uint32)
    absmax = _f32(absmax)
    C = cnt.shape[0]
    state = _f32(s_prev).copy() if s_prev is not None else np.zeros(C, np.float32)
    cls = np.empty(C, np.uint8)
    lib().dai8o_classify_clip(_p(cnt), _p(absmax), C, ctypes.c_int64(M), ctypes.c_float(lam),
                              ctypes.c_float(k), ctypes.c_float(A), _p(state),
                              int(s_prev is not None), _p(cls))
    return state, cls


def grad_scales(g, mode: str = "full", s_prev=None, lam: float = 0.3, k: float = 1.0, A: float = 0.8):
    """Clip values s[C] and classes cls[C] of the per-channel codes under one of the quantization
    strategies of the ablation study (Sec. 4.1), composed from the steps above:
      "full"       Algorithm 1: per-channel sigma, density, discriminator (Eq. 15), clip rule (Eq. 11 / 14)
      "gq"         global quantization: |g|max of the layer for every channel, no clipping
      "gvq_max"    per-channel |g|max, no discriminator, no clipping
      "layer_mcs"  Eq. 15 and Eq. 14 on the statistics of the whole layer (the layer as ONE channel of
                   N*C*H*W elements), one clip value for every channel; s_prev: its previous value
    Returns (s[C] fp32, cls[C] uint8, |g|max of the layer)."""
    g = _f32(g)
    N, C, H, W = g.shape
    absmax, _, sigma, gl = channel_stats(g)
    if mode == "full":
        s, cls = classify_clip(density_count(g, sigma), absmax, N * H * W, s_prev=s_prev, lam=lam, k=k, A=A)
    elif mode == "gq":
        s, cls = np.full(C, gl, np.float32), np.ones(C, np.uint8)
    elif mode == "gvq_max":
        s, cls = absmax.copy(), np.ones(C, np.uint8)
    elif mode == "layer_mcs":
        one = g.reshape(1, 1, N * C * H, W)
        am1, _, sg1, _ = channel_stats(one)
        prev = None if s_prev is None else np.atleast_1d(_f32(s_prev))[:1]
        s1, c1 = classify_clip(density_count(one, sg1), am1, N * C * H * W, s_prev=prev, lam=lam, k=k, A=A)
        s, cls = np.full(C, s1[0], np.float32), np.full(C, c1[0], np.uint8)
    else:
        raise ValueError(mode)
    return s, cls, gl


def rand_uniform(seed: int, stream: int, index: int) -> float:
    return float(lib().dai8o_rand_uniform(seed & 0xFFFFFFFF, stream, index))


def rand_bits(seed: int, stream: int, index: int) -> int:
    return int(lib().dai8o_rand_bits(seed & 0xFFFFFFFF, stream, index))


def quantize(x, scale, stochastic: bool = False, seed: int = 0, stream: int = 0, first_image: int = 0) -> np.ndarray:
    """Eq. 1.  scale: scalar (layer-wide) or array [C] (per channel).  Returns NCHW int8 codes.
    x may be images first_image .. first_image + N - 1 of a larger tensor: stochastic rounding draws
    its numbers by the element's index in the whole tensor."""
    x = _f32(x)
    N, C, H, W = x.shape
    scale = np.atleast_1d(_f32(scale))
    per_channel = scale.shape[0] != 1
    if per_channel:
        assert scale.shape == (C,)
    q = np.empty(x.shape, np.int8)
    lib().dai8o_quantize_at(_p(x), N, C, H, W, ctypes.c_int64(first_image), _p(scale), int(per_channel),
                            int(stochastic), ctypes.c_uint32(seed & 0xFFFFFFFF), ctypes.c_uint32(stream), _p(q))
    return q


def dequantize(q, scale) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int8)
    N, C, H, W = q.shape
    scale = np.atleast_1d(_f32(scale))
    out = np.empty(q.shape, np.float32)
    lib().dai8o_dequantize(_p(q), N, C, H, W, _p(scale), int(scale.shape[0] != 1), _p(out))
    return out


def _geom(N, Cin, Cout, H, W, R, S, stride, pad) -> np.ndarray:
    sh, sw = (stride, stride) if np.isscalar(stride) else stride
    ph, pw = (pad, pad) if np.isscalar(pad) else pad
    return np.array([N, Cin, Cout, H, W, R, S, sh, sw, ph, pw], dtype=np.int32)


def out_hw(H, W, R, S, stride, pad):
    sh, sw = (stride, stride) if np.isscalar(stride) else stride
    ph, pw = (pad, pad) if np.isscalar(pad) else pad
    return (H + 2 * ph - R) // sh + 1, (W + 2 * pw - S) // sw + 1


def _idx(idx):
    if idx is None:
        return None, 0
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    return idx, idx.shape[0]


def conv_fwd_acc(qX, qW, stride=1, pad=0, idx=None):
    """Integer forward convolution.  Returns (acc int64, n_overflow).  acc is (N,Cout,P,Q), or one
    value per flat NCHW output index in ``idx``."""
    qX = np.ascontiguousarray(qX, dtype=np.int8)
    qW = np.ascontiguousarray(qW, dtype=np.int8)
    N, Cin, H, W = qX.shape
    Cout, Cin2, R, S = qW.shape
    assert Cin == Cin2
    P, Q = out_hw(H, W, R, S, stride, pad)
    g = _geom(N, Cin, Cout, H, W, R, S, stride, pad)
    idx, n = _idx(idx)
    acc = np.empty(n if n else (N, Cout, P, Q), np.int64)
    ov = lib().dai8o_conv_fwd_acc(_p(qX), _p(qW), _p(g), _p(idx) if n else None,
                                  ctypes.c_int64(n), _p(acc))
    return acc, int(ov)


def conv_bwd_data_acc(qG, qW, in_hw, stride=1, pad=0, idx=None):
    """Integer input gradient (Eq. 3).  qG is (N,Cout,P,Q); returns acc (N,Cin,H,W) or samples."""
    qG = np.ascontiguousarray(qG, dtype=np.int8)
    qW = np.ascontiguousarray(qW, dtype=np.int8)
    N, Cout, P, Q = qG.shape
    Cout2, Cin, R, S = qW.shape
    assert Cout == Cout2
    H, W = in_hw
    assert (P, Q) == out_hw(H, W, R, S, stride, pad)
    g = _geom(N, Cin, Cout, H, W, R, S, stride, pad)
    idx, n = _idx(idx)
    acc = np.empty(n if n else (N, Cin, H, W), np.int64)
    ov = lib().dai8o_conv_bwd_data_acc(_p(qG), _p(qW), _p(g), _p(idx) if n else None,
                                       ctypes.c_int64(n), _p(acc))
    return acc, int(ov)


def conv_bwd_filter_acc(qX, qG, filter_hw, stride=1, pad=0, idx=None):
    """Integer weight gradient (Eq. 4).  Returns acc (Cout,Cin,R,S) or samples."""
    qX = np.ascontiguousarray(qX, dtype=np.int8)
    qG = np.ascontiguousarray(qG, dtype=np.int8)
    N, Cin, H, W = qX.shape
    N2, Cout, P, Q = qG.shape
    R, S = filter_hw
    assert N == N2 and (P, Q) == out_hw(H, W, R, S, stride, pad)
    g = _geom(N, Cin, Cout, H, W, R, S, stride, pad)
    idx, n = _idx(idx)
    acc = np.empty(n if n else (Cout, Cin, R, S), np.int64)
    ov = lib().dai8o_conv_bwd_filter_acc(_p(qX), _p(qG), _p(g), _p(idx) if n else None,
                                         ctypes.c_int64(n), _p(acc))
    return acc, int(ov)


def _t3(v):
    return (v, v, v) if np.isscalar(v) else tuple(v)


def out_dhw(D, H, W, T, R, S, stride, pad):
    st, pd = _t3(stride), _t3(pad)
    return tuple((n + 2 * p - k) // s + 1 for n, k, s, p in zip((D, H, W), (T, R, S), st, pd))


def conv3_acc(op: str, a, b, geom, idx=None):
    """Integer convolution with a depth dimension and channel groups (3-D convolution, Sec. 4.4; depth-wise
    convolution, Sec. 4.2).  geom = (N, Cin, Cout, D, H, W, T, R, S, stride, pad, groups), stride / pad
    scalars or (d, h, w).  op "fwd": a = X (N,Cin,D,H,W), b = W (Cout,Cin/groups,T,R,S) -> Y (N,Cout,Do,P,Q);
    "bwd_data": a = G, b = W -> dX; "bwd_filter": a = X, b = G -> dW.  Returns (acc int64, n_overflow)."""
    N, Cin, Cout, D, H, W, T, R, S, stride, pad, groups = geom
    st, pd = _t3(stride), _t3(pad)
    Do, P, Q = out_dhw(D, H, W, T, R, S, st, pd)
    g = np.array([N, Cin, Cout, D, H, W, T, R, S, *st, *pd, groups], dtype=np.int32)
    a = np.ascontiguousarray(a, dtype=np.int8)
    b = np.ascontiguousarray(b, dtype=np.int8)
    code = {"fwd": 0, "bwd_data": 1, "bwd_filter": 2}[op]
    shapes = {0: (N, Cout, Do, P, Q), 1: (N, Cin, D, H, W), 2: (Cout, Cin // groups, T, R, S)}
    want_a = {0: (N, Cin, D, H, W), 1: (N, Cout, Do, P, Q), 2: (N, Cin, D, H, W)}[code]
    want_b = {0: (Cout, Cin // groups, T, R, S), 1: (Cout, Cin // groups, T, R, S), 2: (N, Cout, Do, P, Q)}[code]
    assert a.shape == want_a and b.shape == want_b, (a.shape, want_a, b.shape, want_b)
    idx, n = _idx(idx)
    acc = np.empty(n if n else shapes[code], np.int64)
    ov = lib().dai8o_conv3_acc(code, _p(a), _p(b), _p(g), _p(idx) if n else None, ctypes.c_int64(n), _p(acc))
    return acc, int(ov)


def dequant_acc(acc, sa: float, sb) -> np.ndarray:
    """out = float(acc) * ((sa/127) * (sb/127)); sb scalar, or one value per leading index of acc."""
    acc = np.ascontiguousarray(acc, dtype=np.int64)
    sb = np.atleast_1d(_f32(sb))
    per_row = sb.shape[0] != 1
    rows = acc.shape[0] if per_row else 1
    cols = acc.size // rows
    if per_row:
        assert sb.shape[0] == rows
    out = np.empty(acc.shape, np.float32)
    lib().dai8o_dequant_acc(_p(acc), ctypes.c_int64(rows), ctypes.c_int64(cols),
                            ctypes.c_float(sa), _p(sb), int(per_row), _p(out))
    return out
