"""ctypes binding of libmxnorm.so: same names as the C ABI, argument marshalling only.

Every step of the hot path runs in the CUDA kernels behind the C ABI; this module only turns
torch CUDA tensors into device pointers and sizes.  There is no CPU fallback: if the compiled
library is missing the import of this module fails.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmxnorm.so")

ROUND_RCEIL_POW2, ROUND_FLOOR_OCP, ROUND_RCEIL_MAX = 0, 1, 2
SCALES_ROWMAJOR, SCALES_SWIZZLE_128x4 = 0, 1
OK = 0

EXPORTS = ("mxn_scale_bytes", "mxn_status_string", "mx_cast", "rmsnorm_mxfp8_fwd", "mxnorm_fwd",
           "mxnorm_nvfp4_fwd", "mxnorm_bwd", "mxnorm_bwd_workspace_bytes", "mxnorm_fwd_host",
           "mxnorm_fwd_host_workspace_bytes", "mxnorm_bwd_noalloc", "mxnorm_bwd_noalloc_max_scratch_bytes",
           "mxn_device_timeouts", "mxn_device_timeouts_reset", "mxn_selftest_bounded_wait", "mx_cast_fp4", "rmsnorm_mxfp4_fwd", "mxnorm_mxfp4_fwd",
           "mx_cast_transposed", "rmsnorm_nvfp4_fwd", "mxn_selftest_division", "mxn_selftest_dispatch",
           "mx_cast_e5m2", "mx_cast_transposed_e5m2", "mxnorm_postround_fwd",
           "mxnorm_add_fwd", "mx_cast_nvfp4")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2603_13180_b200.build` "
        "(the MXNorm path has no fallback implementation)")

lib = ctypes.CDLL(LIB_PATH)

_vp, _i64, _i32, _f32, _sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
lib.mxn_scale_bytes.argtypes = [_i64, _i64, _i32]
lib.mxn_scale_bytes.restype = _sz
lib.mxn_status_string.argtypes = [_i32]
lib.mxn_status_string.restype = ctypes.c_char_p
lib.mxn_device_timeouts.argtypes = [ctypes.POINTER(ctypes.c_uint)]
lib.mxn_device_timeouts.restype = _i32
lib.mxn_device_timeouts_reset.argtypes = []
lib.mxn_device_timeouts_reset.restype = _i32
lib.mxn_selftest_bounded_wait.argtypes = [ctypes.c_uint, _vp]
lib.mxn_selftest_bounded_wait.restype = _i32
lib.mxn_selftest_division.argtypes = [ctypes.POINTER(ctypes.c_ulonglong)]
lib.mxn_selftest_division.restype = _i32
lib.mxn_selftest_dispatch.argtypes = [_i64, ctypes.POINTER(ctypes.c_longlong), ctypes.POINTER(_i64), ctypes.POINTER(_i32)]
lib.mxn_selftest_dispatch.restype = _i32
lib.mx_cast.argtypes = [_vp, _i64, _i64, _i32, _vp, _vp, _i32, _i32, _vp]
lib.rmsnorm_mxfp8_fwd.argtypes = [_vp, _vp, _i64, _i64, _i32, _f32, _vp, _vp, _vp, _i32, _i32, _vp]
lib.mxnorm_fwd.argtypes = [_vp, _vp, _i64, _i64, _i32, _i32, _f32, _f32, _vp, _vp, _vp, _i32, _i32, _vp]
lib.mxnorm_nvfp4_fwd.argtypes = [_vp, _i64, _i64, _i32, _f32, _f32, _f32, _vp, _vp, _vp, _i32, _vp]
lib.mxnorm_bwd.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _vp, _i32, _vp, _vp, _sz, _vp]
lib.mxnorm_bwd_workspace_bytes.argtypes = [_i64, _i64]
lib.mxnorm_bwd_workspace_bytes.restype = _sz
lib.mxnorm_fwd_host.argtypes = [_vp, _i64, _i64, _i32, _i32, _f32, _f32, _vp, _vp, _vp, _i32, _i32, _vp, _sz, _vp]
lib.mxnorm_fwd_host_workspace_bytes.argtypes = [_i64, _i64, _i32, _i32]
lib.mxnorm_fwd_host_workspace_bytes.restype = _sz
lib.mx_cast_fp4.argtypes = [_vp, _i64, _i64, _i32, _vp, _vp, _i32, _vp]
lib.rmsnorm_mxfp4_fwd.argtypes = [_vp, _i64, _i64, _i32, _f32, _vp, _vp, _vp, _i32, _vp]
lib.mxnorm_mxfp4_fwd.argtypes = [_vp, _i64, _i64, _i32, _i32, _f32, _f32, _vp, _vp, _vp, _i32, _vp]
lib.mxnorm_add_fwd.argtypes = [_vp, _vp, _i64, _i64, _i32, _i32, _f32, _f32, _vp, _vp, _vp, _vp, _i32, _vp]
lib.mxnorm_postround_fwd.argtypes = [_vp, _i64, _i64, _i32, _f32, _vp, _vp, _vp, _i32, _vp]
lib.mx_cast_e5m2.argtypes = [_vp, _i64, _i64, _i32, _vp, _vp, _i32, _vp]
lib.mx_cast_transposed_e5m2.argtypes = [_vp, _i64, _i64, _vp, _vp, _i32, _vp]
lib.rmsnorm_nvfp4_fwd.argtypes = [_vp, _i64, _i64, _f32, _f32, _vp, _vp, _vp, _i32, _vp]
lib.mx_cast_nvfp4.argtypes = [_vp, _i64, _i64, _f32, _vp, _vp, _i32, _vp]
lib.mx_cast_transposed.argtypes = [_vp, _vp, _i64, _i64, _f32, _vp, _vp, _i32, _i32, _vp]
lib.mxnorm_bwd_noalloc.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _vp, _i32, _vp, _vp]
lib.mxnorm_bwd_noalloc_max_scratch_bytes.argtypes = []
lib.mxnorm_bwd_noalloc_max_scratch_bytes.restype = _sz
for _name in ("mx_cast", "rmsnorm_mxfp8_fwd", "mxnorm_fwd", "mxnorm_nvfp4_fwd", "mxnorm_bwd", "mxnorm_fwd_host",
              "mxnorm_bwd_noalloc", "mx_cast_fp4", "rmsnorm_mxfp4_fwd", "mxnorm_mxfp4_fwd",
           "mx_cast_transposed", "rmsnorm_nvfp4_fwd", "mxn_selftest_division", "mxn_selftest_dispatch",
           "mx_cast_e5m2", "mx_cast_transposed_e5m2", "mxnorm_postround_fwd",
           "mxnorm_add_fwd", "mx_cast_nvfp4"):
    getattr(lib, _name).restype = _i32


class MXNormError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def status_string(status: int) -> str:
    return lib.mxn_status_string(status).decode()


def _check(status: int, where: str):
    if status != OK:
        raise MXNormError(status, where)


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _dev(t: torch.Tensor, dtype, name: str):
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise ValueError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t


def device_timeouts() -> int:
    """Synchronises the device and returns how many bounded device-side waits have run out (0 = healthy)."""
    n = ctypes.c_uint(0)
    st = lib.mxn_device_timeouts(ctypes.byref(n))
    if st not in (OK, 7):
        raise MXNormError(st, "mxn_device_timeouts")
    return int(n.value)


def device_timeouts_reset() -> None:
    """Synchronises the device and sets the count of run-out waits back to 0."""
    _check(lib.mxn_device_timeouts_reset(), "mxn_device_timeouts_reset")


def selftest_bounded_wait(polls: int = 2000, stream=None) -> None:
    """Enqueues one warp whose bounded wait (on a barrier nobody completes) must run out after `polls` polls."""
    _check(lib.mxn_selftest_bounded_wait(polls, _stream(stream)), "mxn_selftest_bounded_wait")


def selftest_division() -> int:
    """Re-checks on the current device that the division shortcuts of the NVFP4 kernels equal IEEE division;
    returns the number of mismatching quotients (0)."""
    n = ctypes.c_ulonglong(0)
    _check(lib.mxn_selftest_division(ctypes.byref(n)), "mxn_selftest_division")
    return int(n.value)


def selftest_dispatch(max_D: int = 65536):
    """Host only: (number of accepted forward shapes and options without a compiled kernel, first such D, its case
    code); the count is expected to be 0."""
    n, d, c = ctypes.c_longlong(0), _i64(0), _i32(0)
    _check(lib.mxn_selftest_dispatch(max_D, ctypes.byref(n), ctypes.byref(d), ctypes.byref(c)), "mxn_selftest_dispatch")
    return int(n.value), int(d.value), int(c.value)


def scale_bytes(T: int, K: int, layout: int = SCALES_ROWMAJOR) -> int:
    return int(lib.mxn_scale_bytes(T, K, layout))


def alloc_outputs(T: int, D: int, block: int = 32, layout: int = SCALES_ROWMAJOR, nvfp4: bool = False,
                  device="cuda"):
    """Allocates (codes, scales, rms) for one forward call (torch owns the memory)."""
    codes = torch.empty((T, D // 2 if nvfp4 else D), dtype=torch.uint8, device=device)
    scales = torch.empty((scale_bytes(T, D // block, layout),), dtype=torch.uint8, device=device)
    rms = torch.empty((T,), dtype=torch.float32, device=device)
    return codes, scales, rms


def mx_cast(x, codes, scales, block=32, round=ROUND_RCEIL_POW2, layout=SCALES_ROWMAJOR, stream=None):
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.mx_cast(_ptr(x), T, D, block, _ptr(codes), _ptr(scales), round, layout, _stream(stream)), "mx_cast")


def rmsnorm_mxfp8_fwd(x, gain, codes, scales, rms_out=None, eps=0.0, block=32, round=ROUND_RCEIL_POW2,
                      layout=SCALES_ROWMAJOR, stream=None):
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.rmsnorm_mxfp8_fwd(_ptr(x), _ptr(gain), T, D, block, eps, _ptr(codes), _ptr(scales), _ptr(rms_out),
                                 round, layout, _stream(stream)), "rmsnorm_mxfp8_fwd")


def mxnorm_fwd(x, gain, codes, scales, rms_est_out=None, p=2, coef=0.0, eps=0.0, block=32,
               round=ROUND_RCEIL_POW2, layout=SCALES_ROWMAJOR, stream=None):
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.mxnorm_fwd(_ptr(x), _ptr(gain), T, D, block, p, coef, eps, _ptr(codes), _ptr(scales),
                          _ptr(rms_est_out), round, layout, _stream(stream)), "mxnorm_fwd")


def mxnorm_nvfp4_fwd(x, codes_packed, scales_e4m3, rms_est_out=None, p=2, coef=0.0, eps=0.0, global_scale=1.0,
                     layout=SCALES_ROWMAJOR, stream=None):
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.mxnorm_nvfp4_fwd(_ptr(x), T, D, p, coef, eps, global_scale, _ptr(codes_packed), _ptr(scales_e4m3),
                                _ptr(rms_est_out), layout, _stream(stream)), "mxnorm_nvfp4_fwd")


def mxnorm_bwd_workspace_bytes(T: int, D: int) -> int:
    return int(lib.mxnorm_bwd_workspace_bytes(T, D))


def mxnorm_bwd(x, grad_out, gain, rms, dx, dgain=None, workspace=None, stream=None):
    _dev(x, torch.bfloat16, "x")
    _dev(grad_out, torch.bfloat16, "grad_out")
    T, D = x.shape
    if dx.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("dx must be bf16 or fp32")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.mxnorm_bwd(_ptr(x), _ptr(grad_out), _ptr(gain), _ptr(rms), T, D, _ptr(dx),
                          1 if dx.dtype == torch.float32 else 0, _ptr(dgain), _ptr(workspace), ws_bytes,
                          _stream(stream)), "mxnorm_bwd")


def mxnorm_fwd_host_workspace_bytes(T: int, D: int, block: int = 32, layout: int = SCALES_ROWMAJOR) -> int:
    return int(lib.mxnorm_fwd_host_workspace_bytes(T, D, block, layout))


def mxnorm_fwd_host(x_host, codes_host, scales_host, rms_est_host, workspace, p=2, coef=0.0, eps=0.0, block=32,
                    round=ROUND_RCEIL_POW2, layout=SCALES_ROWMAJOR, stream=None):
    """Host tensors in and out (pin them for asynchronous copies); `workspace` is a CUDA uint8 tensor."""
    if x_host.is_cuda or codes_host.is_cuda or scales_host.is_cuda or x_host.dtype != torch.bfloat16:
        raise ValueError("mxnorm_fwd_host takes host tensors (bf16 input)")
    T, D = x_host.shape
    _check(lib.mxnorm_fwd_host(_ptr(x_host), T, D, block, p, coef, eps, _ptr(codes_host), _ptr(scales_host),
                               _ptr(rms_est_host), round, layout, _ptr(workspace),
                               workspace.numel() * workspace.element_size(), _stream(stream)), "mxnorm_fwd_host")


def mxnorm_bwd_noalloc(x, grad_out, gain, rms, dx, dgain=None, stream=None):
    """mxnorm_bwd for callers that cannot allocate a workspace: the dgain partial sums use an 8 MiB array
    built into the library (shared by all calls on the device - do not overlap two calls).  Raises
    MXNormError(MXN_ERR_TOO_LARGE) when the problem would need more scratch than that."""
    _dev(x, torch.bfloat16, "x")
    _dev(grad_out, torch.bfloat16, "grad_out")
    T, D = x.shape
    if dx.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("dx must be bf16 or fp32")
    _check(lib.mxnorm_bwd_noalloc(_ptr(x), _ptr(grad_out), _ptr(gain), _ptr(rms), T, D, _ptr(dx),
                                  1 if dx.dtype == torch.float32 else 0, _ptr(dgain), _stream(stream)),
           "mxnorm_bwd_noalloc")


def mx_cast_fp4(x, codes_packed, scales, block=32, layout=SCALES_ROWMAJOR, stream=None):
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.mx_cast_fp4(_ptr(x), T, D, block, _ptr(codes_packed), _ptr(scales), layout, _stream(stream)), "mx_cast_fp4")


def rmsnorm_mxfp4_fwd(x, codes_packed, scales, rms_out=None, eps=0.0, block=32, layout=SCALES_ROWMAJOR, stream=None):
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.rmsnorm_mxfp4_fwd(_ptr(x), T, D, block, eps, _ptr(codes_packed), _ptr(scales), _ptr(rms_out), layout,
                                 _stream(stream)), "rmsnorm_mxfp4_fwd")


def mxnorm_mxfp4_fwd(x, codes_packed, scales, rms_est_out=None, p=2, coef=0.0, eps=0.0, block=32,
                     layout=SCALES_ROWMAJOR, stream=None):
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.mxnorm_mxfp4_fwd(_ptr(x), T, D, block, p, coef, eps, _ptr(codes_packed), _ptr(scales), _ptr(rms_est_out),
                                layout, _stream(stream)), "mxnorm_mxfp4_fwd")


def mx_cast_transposed(x, rms, codes_t, scales_t, eps=0.0, round=ROUND_RCEIL_POW2, layout=SCALES_ROWMAJOR, stream=None):
    """Column-wise MXCast of x * (1 / (rms + eps)) (rms may be None): codes_t [D, T], scales_t [D, T/32]."""
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.mx_cast_transposed(_ptr(x), _ptr(rms), T, D, eps, _ptr(codes_t), _ptr(scales_t), round, layout,
                                  _stream(stream)), "mx_cast_transposed")


def rmsnorm_nvfp4_fwd(x, codes_packed, scales_e4m3, rms_out=None, eps=0.0, global_scale=1.0, layout=SCALES_ROWMAJOR,
                      stream=None):
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.rmsnorm_nvfp4_fwd(_ptr(x), T, D, eps, global_scale, _ptr(codes_packed), _ptr(scales_e4m3), _ptr(rms_out),
                                 layout, _stream(stream)), "rmsnorm_nvfp4_fwd")


def mx_cast_nvfp4(x, codes_packed, scales_e4m3, global_scale=1.0, layout=SCALES_ROWMAJOR, stream=None):
    """NVFP4 cast without a normaliser (e.g. of a weight): E2M1 codes two per byte, E4M3 scales per 16 elements."""
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.mx_cast_nvfp4(_ptr(x), T, D, global_scale, _ptr(codes_packed), _ptr(scales_e4m3), layout, _stream(stream)),
           "mx_cast_nvfp4")


def mx_cast_e5m2(x, codes, scales, block=32, layout=SCALES_ROWMAJOR, stream=None):
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.mx_cast_e5m2(_ptr(x), T, D, block, _ptr(codes), _ptr(scales), layout, _stream(stream)), "mx_cast_e5m2")


def mx_cast_transposed_e5m2(x, codes_t, scales_t, layout=SCALES_ROWMAJOR, stream=None):
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.mx_cast_transposed_e5m2(_ptr(x), T, D, _ptr(codes_t), _ptr(scales_t), layout, _stream(stream)),
           "mx_cast_transposed_e5m2")


def mxnorm_postround_fwd(x, codes, scales, rms_est_out=None, eps=0.0, block=32, layout=SCALES_ROWMAJOR, stream=None):
    """MXNorm with the RMS estimated from power-of-two-rounded block absmaxes (the paper's ablation)."""
    _dev(x, torch.bfloat16, "x")
    T, D = x.shape
    _check(lib.mxnorm_postround_fwd(_ptr(x), T, D, block, eps, _ptr(codes), _ptr(scales), _ptr(rms_est_out), layout,
                                    _stream(stream)), "mxnorm_postround_fwd")


def mxnorm_add_fwd(x, residual, h_out, codes, scales, rms_est_out=None, p=2, coef=0.0, eps=0.0, block=32,
                   layout=SCALES_ROWMAJOR, stream=None):
    """h_out = bf16(x + residual) and MXNorm(h_out) in one pass (h_out may be x or residual itself)."""
    _dev(x, torch.bfloat16, "x")
    _dev(residual, torch.bfloat16, "residual")
    T, D = x.shape
    _check(lib.mxnorm_add_fwd(_ptr(x), _ptr(residual), T, D, block, p, coef, eps, _ptr(h_out), _ptr(codes), _ptr(scales),
                              _ptr(rms_est_out), layout, _stream(stream)), "mxnorm_add_fwd")
