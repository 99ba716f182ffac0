"""Helpers for the GPU parity tests: run the CUDA path through the C-ABI binding and compare with
the CPU oracle on the same bf16 bits."""
import numpy as np
import torch

from paper_2603_13180_b200 import workloads as wl

CANARY = 0xA5
GUARD = 256   # guard bytes on both sides of every output buffer


def guarded(nbytes: int, device="cuda"):
    """uint8 buffer of nbytes with canary-filled guard bands; returns (full, view)."""
    full = torch.full((GUARD + nbytes + GUARD,), CANARY, dtype=torch.uint8, device=device)
    return full, full[GUARD:GUARD + nbytes]


def guards_intact(full: torch.Tensor, nbytes: int) -> bool:
    return bool((full[:GUARD] == CANARY).all().item() and (full[GUARD + nbytes:] == CANARY).all().item())


def unswizzle(scales_flat: np.ndarray, T: int, K: int, oracle) -> np.ndarray:
    return scales_flat[oracle.swizzle_index_map(T, K)]


def swizzle_padding_is_zero(scales_flat: np.ndarray, T: int, K: int, oracle) -> bool:
    mask = np.ones(scales_flat.shape, bool)
    mask[oracle.swizzle_index_map(T, K).ravel()] = False
    return bool(np.all(scales_flat[mask] == 0))


def run_fwd(binding, oracle, kind, x_bits, gain_bits=None, *, block=32, p=2, coef=0.0, eps=0.0, round=0,
            layout=0, global_scale=1.0):
    """Runs one forward entry point on the GPU with guard-banded, pre-poisoned outputs.
    Returns (codes [T, cols] u8, scales [T, K] u8 (un-tiled), rms [T] f32 or None)."""
    T, D = x_bits.shape
    x = wl.from_bits(x_bits).cuda()
    gain = None if gain_bits is None else wl.from_bits(gain_bits).cuda()
    nvfp4 = kind in ("nvfp4", "rms_nvfp4", "cast_nvfp4")
    fp4 = nvfp4 or kind in ("cast4", "rms4", "mx4")     # E2M1 codes: two elements per byte
    B = 16 if nvfp4 else block
    K = D // B
    ccols = D // 2 if fp4 else D
    cfull, codes = guarded(T * ccols)
    sbytes = binding.scale_bytes(T, K, layout)
    sfull, scales = guarded(sbytes)
    rfull, rbytes = guarded(T * 4)
    rms = rbytes.view(torch.float32)
    codes.fill_(0x5A)
    scales.fill_(0x5A)
    if kind == "cast":
        binding.mx_cast(x, codes, scales, block=B, round=round, layout=layout)
        rms = None
    elif kind == "rms":
        binding.rmsnorm_mxfp8_fwd(x, gain, codes, scales, rms, eps=eps, block=B, round=round, layout=layout)
    elif kind == "mx":
        binding.mxnorm_fwd(x, gain, codes, scales, rms, p=p, coef=coef, eps=eps, block=B, round=round, layout=layout)
    elif kind == "nvfp4":
        binding.mxnorm_nvfp4_fwd(x, codes, scales, rms, p=p, coef=coef, eps=eps, global_scale=global_scale,
                                 layout=layout)
    elif kind == "postround":
        binding.mxnorm_postround_fwd(x, codes, scales, rms, eps=eps, block=B, layout=layout)
    elif kind == "rms_nvfp4":
        binding.rmsnorm_nvfp4_fwd(x, codes, scales, rms, eps=eps, global_scale=global_scale, layout=layout)
    elif kind == "cast_nvfp4":
        binding.mx_cast_nvfp4(x, codes, scales, global_scale=global_scale, layout=layout)
        rms = None
    elif kind == "cast4":
        binding.mx_cast_fp4(x, codes, scales, block=B, layout=layout)
        rms = None
    elif kind == "rms4":
        binding.rmsnorm_mxfp4_fwd(x, codes, scales, rms, eps=eps, block=B, layout=layout)
    elif kind == "mx4":
        binding.mxnorm_mxfp4_fwd(x, codes, scales, rms, p=p, coef=coef, eps=eps, block=B, layout=layout)
    else:
        raise ValueError(kind)
    torch.cuda.synchronize()
    assert binding.device_timeouts() == 0, "a bounded device-side wait ran out"
    assert guards_intact(cfull, T * ccols) and guards_intact(sfull, sbytes) and guards_intact(rfull, T * 4), \
        "a kernel wrote outside its output buffer"
    codes_np = codes.cpu().numpy().reshape(T, ccols)
    s_np = scales.cpu().numpy()
    if layout == 1:
        assert swizzle_padding_is_zero(s_np, T, K, oracle), "tiled scale padding must be zero"
        s_np = unswizzle(s_np, T, K, oracle)
    else:
        s_np = s_np.reshape(T, K)
    return codes_np, s_np, (None if rms is None else rms.cpu().numpy())


def run_ref(oracle, kind, x_bits, gain_bits=None, *, block=32, p=2, coef=0.0, eps=0.0, round=0, global_scale=1.0):
    if kind == "cast":
        c, s = oracle.mx_cast_ref(x_bits, block=block, mode=round)
        return c, s, None
    if kind == "rms":
        return oracle.rmsnorm_mxfp8_ref(x_bits, gain=gain_bits, eps=eps, block=block, mode=round)
    if kind == "mx":
        return oracle.mxnorm_ref(x_bits, gain=gain_bits, p=p, coef=coef, eps=eps, block=block, mode=round)
    if kind == "nvfp4":
        return oracle.mxnorm_nvfp4_ref(x_bits, p=p, coef=coef, eps=eps, global_scale=global_scale)
    if kind == "postround":
        return oracle.mxnorm_postround_ref(x_bits, eps=eps, block=block)
    if kind == "rms_nvfp4":
        return oracle.rmsnorm_nvfp4_ref(x_bits, eps=eps, global_scale=global_scale)
    if kind == "cast_nvfp4":
        c, s = oracle.nvfp4_cast_ref(x_bits, global_scale=global_scale)
        return c, s, None
    if kind == "cast4":
        c, s = oracle.mx_cast_ref(x_bits, block=block, elem=oracle.ELEM_E2M1)
        return c, s, None
    if kind == "rms4":
        return oracle.rmsnorm_mxfp8_ref(x_bits, eps=eps, block=block, elem=oracle.ELEM_E2M1)
    if kind == "mx4":
        return oracle.mxnorm_ref(x_bits, p=p, coef=coef, eps=eps, block=block, elem=oracle.ELEM_E2M1)
    raise ValueError(kind)


def sm_int(codes: np.ndarray) -> np.ndarray:
    """sign-magnitude byte codes -> signed integers whose difference counts code steps"""
    mag = (codes & 0x7F).astype(np.int32)
    return np.where(codes & 0x80, -mag, mag)


def assert_exact(got, want, what=""):
    gc, gs, gr = got
    wc, ws, wr = want
    assert np.array_equal(gs, ws), f"{what}: {np.count_nonzero(gs != ws)} scale bytes differ"
    assert np.array_equal(gc, wc), f"{what}: {np.count_nonzero(gc != wc)} code bytes differ"
    if wr is not None:
        assert np.array_equal(gr.view(np.uint32), wr.view(np.uint32)), f"{what}: rms differs"


def nibble_steps(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """per-element code-step distance of packed E2M1 bytes (two sign-magnitude nibbles per byte)"""
    def sm(n):
        mag = (n & 7).astype(np.int32)
        return np.where(n & 8, -mag, mag)
    lo = np.abs(sm(a & 0xF) - sm(b & 0xF))
    hi = np.abs(sm(a >> 4) - sm(b >> 4))
    return np.stack([lo, hi], axis=-1).reshape(a.shape[0], -1)


def assert_within_rounding_of_rho(got, want, block, what="", fp4=False):
    """Tolerance for a path whose fp32 normalisation factor may round differently from the oracle's
    (the binary32 sum of squares of the RMSNorm baseline): r within 1e-6 relative; scale bytes may
    differ (by one) in at most 1e-6 of the blocks; outside those blocks at most 1e-4 of the codes
    differ and only by one code step."""
    gc, gs, gr = got
    wc, ws, wr = want
    assert np.all(np.abs(gr.astype(np.float64) - wr) <= 1e-6 * np.abs(wr)), f"{what}: rms beyond 1e-6"
    sdiff = gs != ws
    assert sdiff.mean() <= 1e-6 or sdiff.sum() <= 1, f"{what}: {sdiff.sum()} scales differ"
    assert np.all(np.abs(gs.astype(int) - ws.astype(int)) <= 1)
    keep = ~np.repeat(sdiff, block, axis=1)
    d = (nibble_steps(gc, wc) if fp4 else np.abs(sm_int(gc) - sm_int(wc)))[keep]
    assert d.max(initial=0) <= 1, f"{what}: a code differs by more than one step"
    assert (d != 0).mean() <= 1e-4, f"{what}: {(d != 0).mean():.2e} of codes differ"
    return int(sdiff.sum()), int((d != 0).sum())
