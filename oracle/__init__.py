"""CPU oracle for the MXNorm hot path — TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes front end of ``mxnorm_oracle.c`` (plain C, fp64 statistics,
fp32 element arithmetic exactly as the paper's algorithms state them).  It is
independent of the CUDA library: nothing here imports the GPU package and the
GPU package never imports this.  Only the tests, the smoke check and the
benchmark's CPU-baseline legs may use it.

All tensors are numpy arrays on the host; bf16 tensors are ``uint16`` bit
patterns of shape ``[T, D]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mxnorm_oracle.c")
_LIB = os.path.join(_HERE, "libmxnorm_oracle.so")

ROUND_RCEIL_POW2, ROUND_FLOOR_OCP, ROUND_RCEIL_MAX = 0, 1, 2
ELEM_E4M3, ELEM_E2M1, ELEM_E5M2 = 0, 1, 2

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fused multiply-adds, OpenMP over rows)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=gnu11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-fPIC", "-shared", "-Wall", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i64, i32, f32, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_float, ctypes.c_void_p
        lib.mx_cast_ref.argtypes = [vp, i64, i64, i32, i32, i32, vp, vp]
        lib.rmsnorm_mxfp8_ref.argtypes = [vp, vp, i64, i64, i32, f32, i32, i32, vp, vp, vp]
        lib.mxnorm_ref.argtypes = [vp, vp, i64, i64, i32, i32, f32, f32, i32, i32, vp, vp, vp]
        lib.mxnorm_nvfp4_ref.argtypes = [vp, i64, i64, i32, f32, f32, f32, vp, vp, vp]
        lib.mxnorm_bwd_ref.argtypes = [vp, vp, vp, vp, i64, i64, vp, vp]
        lib.rmsnorm_nvfp4_ref.argtypes = [vp, i64, i64, f32, f32, vp, vp, vp]
        lib.rmsnorm_nvfp4_ref.restype = i32
        lib.nvfp4_cast_ref.argtypes = [vp, i64, i64, f32, vp, vp]
        lib.nvfp4_cast_ref.restype = i32
        lib.mxnorm_postround_ref.argtypes = [vp, i64, i64, i32, f32, i32, vp, vp, vp]
        lib.mxnorm_postround_ref.restype = i32
        lib.mxnorm_add_ref.argtypes = [vp, vp, i64, i64, i32, i32, f32, f32, i32, vp, vp, vp, vp]
        lib.mxnorm_add_ref.restype = i32
        lib.mxn_ref_postround_f.argtypes = [ctypes.c_double, i32]
        lib.mxn_ref_postround_f.restype = ctypes.c_double
        lib.mxn_ref_postround_f_inverse.argtypes = [ctypes.c_double, i32]
        lib.mxn_ref_postround_f_inverse.restype = ctypes.c_double
        lib.mxn_ref_postround_estimate.argtypes = [vp, i64, i32, vp]
        lib.mxn_ref_postround_estimate.restype = None
        lib.mx_cast_transposed_ref.argtypes = [vp, vp, i64, i64, i32, f32, i32, i32, vp, vp]
        lib.mx_cast_transposed_ref.restype = i32
        for f in (lib.mx_cast_ref, lib.rmsnorm_mxfp8_ref, lib.mxnorm_ref, lib.mxnorm_nvfp4_ref,
                  lib.mxnorm_bwd_ref):
            f.restype = i32
        lib.mxn_ref_coef.argtypes = [i32, i32]
        lib.mxn_ref_coef.restype = f32
        lib.mxn_ref_swizzle_offset.argtypes = [i64, i64, i64]
        lib.mxn_ref_swizzle_offset.restype = i64
        lib.mxn_ref_swizzle_bytes.argtypes = [i64, i64]
        lib.mxn_ref_swizzle_bytes.restype = i64
        lib.mxn_ref_e4m3_encode.argtypes = [f32]
        lib.mxn_ref_e4m3_encode.restype = ctypes.c_uint8
        lib.mxn_ref_e4m3_decode.argtypes = [ctypes.c_uint8]
        lib.mxn_ref_e4m3_decode.restype = f32
        lib.mxn_ref_e2m1_encode.argtypes = [f32]
        lib.mxn_ref_e2m1_encode.restype = ctypes.c_uint8
        lib.mxn_ref_e5m2_encode.argtypes = [f32]
        lib.mxn_ref_e5m2_encode.restype = ctypes.c_uint8
        lib.mxn_ref_e8m0_scale.argtypes = [f32, i32, i32]
        lib.mxn_ref_e8m0_scale.restype = ctypes.c_uint8
        lib.mxn_ref_num_threads.restype = i32
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _bf16(a, shape_len):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16 and a.ndim == shape_len, (a.dtype, a.shape)
    return a


def _code_cols(D, elem):
    return D // 2 if elem == ELEM_E2M1 else D


def _check(rc, name):
    if rc != 0:
        raise ValueError(f"{name}: oracle rejected the shape/arguments (rc={rc})")


def num_threads() -> int:
    return int(_load().mxn_ref_num_threads())


def coef(block: int, p: int) -> float:
    """The paper's printed correction constant RMS/G_p for (block, p) as fp32."""
    return float(_load().mxn_ref_coef(block, p))


def mx_cast_ref(x, block=32, mode=ROUND_RCEIL_POW2, elem=ELEM_E4M3):
    """MXCast (Section 3.2): returns (codes [T, D or D/2] u8, scales [T, K] u8)."""
    x = _bf16(x, 2)
    T, D = x.shape
    codes = np.zeros((T, _code_cols(D, elem)), np.uint8)
    scales = np.zeros((T, D // block if D % block == 0 else 0), np.uint8)
    _check(_load().mx_cast_ref(_p(x), T, D, block, mode, elem, _p(codes), _p(scales)), "mx_cast_ref")
    return codes, scales


def rmsnorm_mxfp8_ref(x, gain=None, eps=0.0, block=32, mode=ROUND_RCEIL_POW2, elem=ELEM_E4M3):
    """Algorithm 1: returns (codes, scales, rms [T] f32)."""
    x = _bf16(x, 2)
    T, D = x.shape
    g = None if gain is None else _bf16(gain, 1)
    codes = np.zeros((T, _code_cols(D, elem)), np.uint8)
    scales = np.zeros((T, D // block if D % block == 0 else 0), np.uint8)
    rms = np.zeros((T,), np.float32)
    _check(_load().rmsnorm_mxfp8_ref(_p(x), _p(g), T, D, block, eps, mode, elem,
                                     _p(codes), _p(scales), _p(rms)), "rmsnorm_mxfp8_ref")
    return codes, scales, rms


def mxnorm_ref(x, gain=None, p=2, coef=0.0, eps=0.0, block=32, mode=ROUND_RCEIL_POW2,
               elem=ELEM_E4M3):
    """Algorithm 2: returns (codes, scales, rms_estimate [T] f32)."""
    x = _bf16(x, 2)
    T, D = x.shape
    g = None if gain is None else _bf16(gain, 1)
    codes = np.zeros((T, _code_cols(D, elem)), np.uint8)
    scales = np.zeros((T, D // block if D % block == 0 else 0), np.uint8)
    rms = np.zeros((T,), np.float32)
    _check(_load().mxnorm_ref(_p(x), _p(g), T, D, block, p, coef, eps, mode, elem,
                              _p(codes), _p(scales), _p(rms)), "mxnorm_ref")
    return codes, scales, rms


def mxnorm_nvfp4_ref(x, p=2, coef=0.0, eps=0.0, global_scale=1.0):
    """NVFP4 variant: returns (packed codes [T, D/2] u8, E4M3 scales [T, D/16] u8, rms_estimate)."""
    x = _bf16(x, 2)
    T, D = x.shape
    codes = np.zeros((T, D // 2), np.uint8)
    scales = np.zeros((T, D // 16 if D % 16 == 0 else 0), np.uint8)
    rms = np.zeros((T,), np.float32)
    _check(_load().mxnorm_nvfp4_ref(_p(x), T, D, p, coef, eps, global_scale,
                                    _p(codes), _p(scales), _p(rms)), "mxnorm_nvfp4_ref")
    return codes, scales, rms


def rmsnorm_nvfp4_ref(x, eps=0.0, global_scale=1.0):
    """RMSNorm followed by the NVFP4 cast: returns (packed codes [T, D/2] u8, E4M3 scales [T, D/16] u8, rms)."""
    x = _bf16(x, 2)
    T, D = x.shape
    codes = np.zeros((T, D // 2), np.uint8)
    scales = np.zeros((T, D // 16 if D % 16 == 0 else 0), np.uint8)
    rms = np.zeros((T,), np.float32)
    _check(_load().rmsnorm_nvfp4_ref(_p(x), T, D, eps, global_scale, _p(codes), _p(scales), _p(rms)),
           "rmsnorm_nvfp4_ref")
    return codes, scales, rms


def nvfp4_cast_ref(x, global_scale=1.0):
    """Plain NVFP4 cast (no normalisation): returns (packed codes [T, D/2] u8, E4M3 scales [T, D/16] u8)."""
    x = _bf16(x, 2)
    T, D = x.shape
    codes = np.zeros((T, D // 2), np.uint8)
    scales = np.zeros((T, D // 16 if D % 16 == 0 else 0), np.uint8)
    _check(_load().nvfp4_cast_ref(_p(x), T, D, global_scale, _p(codes), _p(scales)), "nvfp4_cast_ref")
    return codes, scales


def mxnorm_add_ref(x, res, p=2, coef=0.0, eps=0.0, block=32, mode=ROUND_RCEIL_POW2):
    """Residual add then MXNorm: returns (h [T, D] bf16 bits, codes, scales, rms_estimate)."""
    x = _bf16(x, 2)
    res = _bf16(res, 2)
    assert x.shape == res.shape
    T, D = x.shape
    h = np.zeros((T, D), np.uint16)
    codes = np.zeros((T, D), np.uint8)
    scales = np.zeros((T, D // block if D % block == 0 else 0), np.uint8)
    rms = np.zeros((T,), np.float32)
    _check(_load().mxnorm_add_ref(_p(x), _p(res), T, D, block, p, coef, eps, mode, _p(h), _p(codes), _p(scales), _p(rms)),
           "mxnorm_add_ref")
    return h, codes, scales, rms


def mxnorm_postround_ref(x, eps=0.0, block=32, mode=ROUND_RCEIL_POW2):
    """Post-round MXNorm (RMS from the power-of-two-rounded block absmaxes): returns (codes, scales, rms_estimate)."""
    x = _bf16(x, 2)
    T, D = x.shape
    codes = np.zeros((T, D), np.uint8)
    scales = np.zeros((T, D // block if D % block == 0 else 0), np.uint8)
    rms = np.zeros((T,), np.float32)
    _check(_load().mxnorm_postround_ref(_p(x), T, D, block, eps, mode, _p(codes), _p(scales), _p(rms)),
           "mxnorm_postround_ref")
    return codes, scales, rms


def postround_f(sigma: float, block: int) -> float:
    return float(_load().mxn_ref_postround_f(sigma, block))


def postround_f_inverse(x: float, block: int) -> float:
    return float(_load().mxn_ref_postround_f_inverse(x, block))


def postround_estimate(xbar, block: int) -> np.ndarray:
    """r~ = f^-1(xbar) through the 64-interval table for an array of arguments (binary64, before the rounding to
    binary32)."""
    xb = np.ascontiguousarray(np.atleast_1d(xbar), dtype=np.float64)
    out = np.zeros_like(xb)
    _load().mxn_ref_postround_estimate(_p(xb), xb.size, block, _p(out))
    return out


def mxnorm_bwd_ref(x, g, gain, rms, want_dx=True, want_dgain=True):
    """Straight-through backward in fp64: returns (dX [T, D] f64 | None, dgain [D] f64 | None)."""
    x = _bf16(x, 2)
    g = _bf16(g, 2)
    T, D = x.shape
    assert g.shape == x.shape
    gn = None if gain is None else _bf16(gain, 1)
    rms = np.ascontiguousarray(rms, dtype=np.float32)
    dx = np.zeros((T, D), np.float64) if want_dx else None
    dg = np.zeros((D,), np.float64) if want_dgain else None
    _check(_load().mxnorm_bwd_ref(_p(x), _p(g), _p(gn), _p(rms), T, D, _p(dx), _p(dg)),
           "mxnorm_bwd_ref")
    return dx, dg


def mx_cast_transposed_ref(x, rms=None, eps=0.0, block=32, mode=ROUND_RCEIL_POW2, elem=ELEM_E4M3):
    """Column-wise MXCast of x * rho (rho = 1/(rms+eps), or 1): returns (codes [D, T] u8, scales [D, T/block] u8)."""
    x = _bf16(x, 2)
    T, D = x.shape
    r = None if rms is None else np.ascontiguousarray(rms, dtype=np.float32)
    codes = np.zeros((D, T), np.uint8)
    scales = np.zeros((D, T // block if T % block == 0 else 0), np.uint8)
    _check(_load().mx_cast_transposed_ref(_p(x), _p(r), T, D, block, eps, mode, elem, _p(codes), _p(scales)),
           "mx_cast_transposed_ref")
    return codes, scales


def swizzle_offset(r: int, c: int, K: int) -> int:
    return int(_load().mxn_ref_swizzle_offset(r, c, K))


def swizzle_bytes(T: int, K: int) -> int:
    return int(_load().mxn_ref_swizzle_bytes(T, K))


def swizzle_index_map(T: int, K: int) -> np.ndarray:
    """[T, K] int64 array of byte offsets into the 128x4-tiled scale buffer (same formula as
    ``swizzle_offset``, evaluated with numpy integer arithmetic for whole tensors)."""
    r = np.arange(T, dtype=np.int64)[:, None]
    c = np.arange(K, dtype=np.int64)[None, :]
    tiles_per_row = (K + 3) // 4
    rr = r % 128
    return ((r // 128) * tiles_per_row + c // 4) * 512 + (rr % 32) * 16 + (rr // 32) * 4 + (c % 4)


def e4m3_encode(q: float) -> int:
    return int(_load().mxn_ref_e4m3_encode(q))


def e4m3_decode(c: int) -> float:
    return float(_load().mxn_ref_e4m3_decode(c))


def e2m1_encode(q: float) -> int:
    return int(_load().mxn_ref_e2m1_encode(q))


def e5m2_encode(q: float) -> int:
    return int(_load().mxn_ref_e5m2_encode(q))


def e8m0_scale(a: float, mode=ROUND_RCEIL_POW2, elem=ELEM_E4M3) -> int:
    return int(_load().mxn_ref_e8m0_scale(a, mode, elem))
