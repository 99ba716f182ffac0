"""Consumer check of the tiled scale layout: the (codes, scales) that mxnorm_fwd and mx_cast emit with
MXN_SCALES_SWIZZLE_128x4 are fed to a block-scaled tensor-core GEMM (cuBLAS through torch._scaled_mm)
and the product is compared with a plain matmul of the dequantised tensors.  This is the MXNormLinear
forward of Section 3.7, H = MXNorm(X) MXCast(W gamma)^T, and it pins the layout formula against the
consumer that defines it."""
import numpy as np
import pytest
import torch

from paper_2603_13180_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _dequant(codes, scales_rowmajor, T, D, elem=torch.float8_e4m3fn):
    K = D // 32
    vals = codes.view(elem).float().view(T, K, 32)
    return (vals * torch.exp2(scales_rowmajor.view(T, K, 1).float() - 127.0)).view(T, D).double()


@pytest.mark.parametrize("T,D,N", [(256, 512, 128), (384, 4096, 256), (200, 1024, 96)])
def test_block_scaled_gemm_consumes_tiled_scales(oracle, T, D, N):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_13180_b200 import binding as mx
    if not hasattr(torch, "_scaled_mm") or not hasattr(torch, "float8_e8m0fnu"):
        pytest.skip("this torch has no block-scaled matmul")
    inp = wl.make_inputs(wl.Workload("t", T, D, seed=T + D, outlier_frac=0.002, has_gain=True))
    x = inp["x"].cuda()
    g = torch.Generator(device="cpu").manual_seed(N)
    w = (0.05 * torch.randn(N, D, generator=g)).to(torch.bfloat16).cuda()
    w_fused = (w.float() * inp["gain"].cuda().float()).to(torch.bfloat16)      # gain folded into the weight (Sec. 3.7)

    cx, sx, _ = mx.alloc_outputs(T, D, 32, mx.SCALES_SWIZZLE_128x4)
    cw, sw, _ = mx.alloc_outputs(N, D, 32, mx.SCALES_SWIZZLE_128x4)
    mx.mxnorm_fwd(x, None, cx, sx, None, eps=1e-5, layout=mx.SCALES_SWIZZLE_128x4)
    mx.mx_cast(w_fused, cw, sw, layout=mx.SCALES_SWIZZLE_128x4)
    try:
        out = torch._scaled_mm(cx.view(torch.float8_e4m3fn), cw.view(torch.float8_e4m3fn).t(),
                               scale_a=sx.view(torch.float8_e8m0fnu), scale_b=sw.view(torch.float8_e8m0fnu),
                               out_dtype=torch.bfloat16)
    except (RuntimeError, NotImplementedError) as e:   # the consumer itself is unavailable in this build
        pytest.skip(f"torch._scaled_mm rejected MXFP8 block scales: {str(e)[:120]}")
    torch.cuda.synchronize()

    # reference: un-tile the scales with the oracle's index map, dequantise, multiply in binary64
    K = D // 32
    sx_rm = torch.from_numpy(sx.cpu().numpy()[oracle.swizzle_index_map(T, K)]).cuda()
    sw_rm = torch.from_numpy(sw.cpu().numpy()[oracle.swizzle_index_map(N, K)]).cuda()
    ref = _dequant(cx, sx_rm, T, D) @ _dequant(cw, sw_rm, N, D).t()
    err = (out.double() - ref).abs().max().item() / ref.abs().max().item()
    assert err < 1e-2, err                      # bf16 output rounding + fp32 accumulation order

    # negative control: the same bytes in row-major order are NOT what the consumer expects
    cx0, sx0, _ = mx.alloc_outputs(T, D, 32, mx.SCALES_ROWMAJOR)
    mx.mxnorm_fwd(x, None, cx0, sx0, None, eps=1e-5, layout=mx.SCALES_ROWMAJOR)
    if T % 128 == 0:
        bad = torch._scaled_mm(cx0.view(torch.float8_e4m3fn), cw.view(torch.float8_e4m3fn).t(),
                               scale_a=sx0.view(torch.float8_e8m0fnu), scale_b=sw.view(torch.float8_e8m0fnu),
                               out_dtype=torch.bfloat16)
        bad_err = (bad.double() - ref).abs().max().item() / ref.abs().max().item()
        assert bad_err > 10 * err


@pytest.mark.parametrize("grad_e5m2", [False, True])
@pytest.mark.parametrize("T,D,N", [(256, 512, 128), (512, 1024, 256), (384, 768, 96)])
def test_weight_gradient_gemm_consumes_the_column_wise_casts(oracle, T, D, N, grad_e5m2):
    """The weight gradient of Section 3.7, grad W = MXCast(grad H^T) MXCast(rho~ X), contracts over the TOKENS: both
    operands are the [*, T] outputs of mx_cast_transposed with their tiled scales, handed to the block-scaled GEMM as
    they are.  Pins the transposed outputs' layout against the consumer."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_13180_b200 import binding as mx
    if not hasattr(torch, "_scaled_mm") or not hasattr(torch, "float8_e8m0fnu"):
        pytest.skip("this torch has no block-scaled matmul")
    tiled = mx.SCALES_SWIZZLE_128x4
    inp = wl.make_inputs(wl.Workload("t", T, D, seed=T + D + N, outlier_frac=0.002))
    x = inp["x"].cuda()
    g = torch.Generator(device="cpu").manual_seed(N)
    grad_h = (1e-2 * torch.randn(T, N, generator=g)).to(torch.bfloat16).cuda()

    # forward: r~ per token; then the two column-wise casts
    cx, sx, rms = mx.alloc_outputs(T, D, 32, tiled)
    mx.mxnorm_fwd(x, None, cx, sx, rms, eps=1e-5, layout=tiled)
    KT = T // 32
    xt = torch.empty((D, T), dtype=torch.uint8, device="cuda")
    xts = torch.empty(mx.scale_bytes(D, KT, tiled), dtype=torch.uint8, device="cuda")
    mx.mx_cast_transposed(x, rms, xt, xts, eps=1e-5, layout=tiled)
    gt = torch.empty((N, T), dtype=torch.uint8, device="cuda")
    gts = torch.empty(mx.scale_bytes(N, KT, tiled), dtype=torch.uint8, device="cuda")
    gdt = torch.float8_e5m2 if grad_e5m2 else torch.float8_e4m3fn       # E5M2: the option the paper names for gradients
    if grad_e5m2:
        mx.mx_cast_transposed_e5m2(grad_h, gt, gts, layout=tiled)
    else:
        mx.mx_cast_transposed(grad_h, None, gt, gts, layout=tiled)
    try:
        out = torch._scaled_mm(gt.view(gdt), xt.view(torch.float8_e4m3fn).t(),
                               scale_a=gts.view(torch.float8_e8m0fnu), scale_b=xts.view(torch.float8_e8m0fnu),
                               out_dtype=torch.bfloat16)
    except (RuntimeError, NotImplementedError) as e:
        pytest.skip(f"torch._scaled_mm rejected these MXFP8 operands: {str(e)[:120]}")
    torch.cuda.synchronize()

    gts_rm = torch.from_numpy(gts.cpu().numpy()[oracle.swizzle_index_map(N, KT)]).cuda()
    xts_rm = torch.from_numpy(xts.cpu().numpy()[oracle.swizzle_index_map(D, KT)]).cuda()
    a, b = _dequant(gt, gts_rm, N, T, gdt), _dequant(xt, xts_rm, D, T)     # [N, T] and [D, T], blocks along T
    ref = a @ b.t()
    err = (out.double() - ref).abs().max().item() / ref.abs().max().item()
    assert err < 1e-2, err
    # and the quantised product is the weight gradient of the unquantised operands to MXFP8 accuracy
    rho = 1.0 / (rms.double() + 1e-5)
    exact = grad_h.double().t() @ (x.double() * rho[:, None])
    assert (ref - exact).abs().max().item() < 0.08 * exact.abs().max().item()


_E2M1 = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def _dequant_nvfp4(codes_packed, scales_rowmajor_e4m3, T, D):
    """[T, D/2] bytes (low nibble = even element) and E4M3 scale bytes [T, D/16] -> [T, D] binary64"""
    lut = torch.tensor(_E2M1 + [-v for v in _E2M1], dtype=torch.float64, device=codes_packed.device)
    lo, hi = (codes_packed & 0xF).long(), (codes_packed >> 4).long()
    vals = torch.stack([lut[lo], lut[hi]], dim=-1).view(T, D // 16, 16)
    sc = scales_rowmajor_e4m3.view(torch.float8_e4m3fn).double().view(T, D // 16, 1)
    return (vals * sc).view(T, D)


@pytest.mark.parametrize("T,D,N", [(256, 512, 128), (384, 4096, 256)])
def test_nvfp4_gemm_consumes_packed_codes_and_e4m3_scales(oracle, T, D, N):
    """NVFP4 (which the paper does not define beyond block 16 / E2M1): the packed nibbles and the tiled E4M3 block scales
    that mxnorm_nvfp4_fwd emits are what the block-scaled FP4 GEMM of the vendor library expects - nibble order, scale
    format and scale layout pinned against that consumer."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_13180_b200 import binding as mx
    if not hasattr(torch, "_scaled_mm") or not hasattr(torch, "float4_e2m1fn_x2"):
        pytest.skip("this torch has no FP4 block-scaled matmul")
    tiled = mx.SCALES_SWIZZLE_128x4
    x = wl.make_inputs(wl.Workload("t", T, D, seed=T + D, outlier_frac=0.002))["x"].cuda()
    w = wl.make_inputs(wl.Workload("w", N, D, seed=N + D))["x"].cuda()
    cx, sx, _ = mx.alloc_outputs(T, D, 16, tiled, nvfp4=True)
    cw, sw, _ = mx.alloc_outputs(N, D, 16, tiled, nvfp4=True)
    mx.mxnorm_nvfp4_fwd(x, cx, sx, None, eps=1e-5, layout=tiled)
    mx.mx_cast_nvfp4(w, cw, sw, layout=tiled)                               # the weight operand: cast without a normaliser
    try:
        out = torch._scaled_mm(cx.view(torch.float4_e2m1fn_x2), cw.view(torch.float4_e2m1fn_x2).t(),
                               scale_a=sx.view(torch.float8_e4m3fn), scale_b=sw.view(torch.float8_e4m3fn),
                               out_dtype=torch.bfloat16)
    except (RuntimeError, NotImplementedError, TypeError) as e:
        pytest.skip(f"torch._scaled_mm rejected NVFP4 operands: {str(e)[:160]}")
    torch.cuda.synchronize()
    K = D // 16
    sx_rm = torch.from_numpy(sx.cpu().numpy()[oracle.swizzle_index_map(T, K)]).cuda()
    sw_rm = torch.from_numpy(sw.cpu().numpy()[oracle.swizzle_index_map(N, K)]).cuda()
    ref = _dequant_nvfp4(cx, sx_rm, T, D) @ _dequant_nvfp4(cw, sw_rm, N, D).t()
    err = (out.double() - ref).abs().max().item() / ref.abs().max().item()
    assert err < 1e-2, err
