"""GPU parity: the CUDA forward kernels (through the C ABI) against the CPU oracle, element by
element on the same seeded bf16 bits."""
import numpy as np
import pytest
import torch

from paper_2603_13180_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_13180_b200 import binding as b
    return b


def rows(T, D, seed, outliers=True):
    w = wl.Workload("t", T, D, seed=seed, outlier_frac=0.002 if outliers else 0.0, has_gain=True)
    inp = wl.make_inputs(w)
    return wl.bits(inp["x"]), wl.bits(inp["gain"])


# shapes: single lane active, ragged K (not a multiple of 32), several passes, rows spanning
# 2/4/8 warps, odd T (ragged last CTA)
SHAPES = [(1, 32), (5, 64), (37, 768), (130, 1024), (9, 2560), (33, 4096), (6, 5120), (5, 8192), (3, 16384),
          (2, 32768), (257, 2048),
          # hidden sizes {3,5,7} * 2^r of the paper's sweep: rows spanning 3, 5, 6 and 7 warps
          (7, 3072), (5, 6144), (4, 7168), (3, 10240), (3, 12288), (3, 14336), (11, 1280), (9, 1792), (10, 1536), (6, 3584), (133, 1280), (130, 2560),
          # several rows per warp (D = 512: four), with a ragged last warp
          (131, 512), (3, 512)]


@pytest.mark.parametrize("T,D", SHAPES)
def test_mxnorm_fwd_matches_oracle_bit_for_bit(binding, oracle, T, D):
    x, gain = rows(T, D, seed=T + D)
    for p in (2, 1):
        for eps in (0.0, 1e-5):
            got = gu.run_fwd(binding, oracle, "mx", x, p=p, eps=eps)
            gu.assert_exact(got, gu.run_ref(oracle, "mx", x, p=p, eps=eps), f"mxnorm p={p} eps={eps} {T}x{D}")
    got = gu.run_fwd(binding, oracle, "mx", x, gain, eps=1e-5)
    gu.assert_exact(got, gu.run_ref(oracle, "mx", x, gain, eps=1e-5), f"mxnorm+gain {T}x{D}")
    got = gu.run_fwd(binding, oracle, "mx", x, coef=0.5, eps=0.0)
    gu.assert_exact(got, gu.run_ref(oracle, "mx", x, coef=0.5, eps=0.0), "mxnorm coef override")


@pytest.mark.parametrize("T,D", SHAPES)
def test_mx_cast_matches_oracle_bit_for_bit(binding, oracle, T, D):
    x, _ = rows(T, D, seed=3 * T + D)
    for rnd in (0, 1, 2):
        got = gu.run_fwd(binding, oracle, "cast", x, round=rnd)
        gu.assert_exact(got, gu.run_ref(oracle, "cast", x, round=rnd), f"mx_cast round={rnd} {T}x{D}")


@pytest.mark.parametrize("T,D", SHAPES)
def test_rmsnorm_mxfp8_fwd_matches_oracle(binding, oracle, T, D):
    x, gain = rows(T, D, seed=5 * T + D)
    for g in (None, gain):
        got = gu.run_fwd(binding, oracle, "rms", x, g, eps=1e-5)
        gu.assert_within_rounding_of_rho(got, gu.run_ref(oracle, "rms", x, g, eps=1e-5), 32, f"rmsnorm {T}x{D}")


@pytest.mark.parametrize("block", [16, 64])
@pytest.mark.parametrize("T,D", [(3, 64), (19, 1024), (5, 2048), (9, 2560), (130, 2560), (6, 3072), (7, 4096), (4, 8192), (3, 16384),
                                 (10, 1536), (6, 3584), (11, 1280), (133, 1280), (37, 768), (131, 512),
                                 # with a gain every block size runs as 16-element pieces: rows of 3, 5, 6, 7 and 16 warps
                                 (3, 5120), (5, 6144), (3, 7168), (2, 10240), (2, 12288), (2, 14336), (2, 32768)])
def test_other_block_sizes(binding, oracle, T, D, block):
    x, gain = rows(T, D, seed=T + D + block)
    got = gu.run_fwd(binding, oracle, "mx", x, block=block, eps=1e-5)
    gu.assert_exact(got, gu.run_ref(oracle, "mx", x, block=block, eps=1e-5), f"mxnorm B={block}")
    got = gu.run_fwd(binding, oracle, "mx", x, block=block, p=1)
    gu.assert_exact(got, gu.run_ref(oracle, "mx", x, block=block, p=1), f"mxnorm p=1 B={block}")
    got = gu.run_fwd(binding, oracle, "cast", x, block=block)
    gu.assert_exact(got, gu.run_ref(oracle, "cast", x, block=block), f"mx_cast B={block}")
    got = gu.run_fwd(binding, oracle, "rms", x, gain, block=block, eps=1e-5)
    gu.assert_within_rounding_of_rho(got, gu.run_ref(oracle, "rms", x, gain, block=block, eps=1e-5), block, "rms")
    for layout in (0, 1):
        got = gu.run_fwd(binding, oracle, "mx", x, gain, block=block, eps=1e-5, layout=layout)
        gu.assert_exact(got, gu.run_ref(oracle, "mx", x, gain, block=block, eps=1e-5), f"mxnorm with gain B={block} layout={layout}")


@pytest.mark.parametrize("T,D", [(41, 2048), (9, 2560), (5, 5120), (3, 12288)])
@pytest.mark.parametrize("rnd", [1, 2])
def test_other_rounding_modes(binding, oracle, rnd, T, D):
    x, gain = rows(T, D, seed=17 + D)
    got = gu.run_fwd(binding, oracle, "mx", x, round=rnd, eps=1e-5)
    gu.assert_exact(got, gu.run_ref(oracle, "mx", x, round=rnd, eps=1e-5), f"mxnorm round={rnd}")
    got = gu.run_fwd(binding, oracle, "mx", x, gain, round=rnd)
    gu.assert_exact(got, gu.run_ref(oracle, "mx", x, gain, round=rnd), f"mxnorm gain round={rnd}")


@pytest.mark.parametrize("T,D", [(1, 32), (37, 768), (128, 128), (200, 192), (300, 4096), (129, 2560), (131, 512)])
def test_tiled_scale_layout(binding, oracle, T, D):
    x, _ = rows(T, D, seed=T * 7 + D)
    for kind in ("mx", "cast", "rms"):
        got = gu.run_fwd(binding, oracle, kind, x, layout=1, eps=1e-5)
        want = gu.run_ref(oracle, kind, x, eps=1e-5)
        if kind == "rms":
            gu.assert_within_rounding_of_rho(got, want, 32, "tiled rms")
        else:
            gu.assert_exact(got, want, f"tiled {kind} {T}x{D}")


def test_all_bf16_bit_patterns(binding, oracle):
    pats = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    pats = pats[(pats & 0x7F80) != 0x7F80]                      # finite values only
    # as lone block maxima (mx_cast sees every exponent/mantissa, zeros, subnormals, the largest values) ...
    x = np.zeros((pats.size, 64), np.uint16)
    x[:, 0] = pats
    x[:, 33] = pats >> 1
    x[(x[:, 33] & 0x7F80) == 0x7F80, 33] = 0
    for rnd in (0, 1, 2):
        gu.assert_exact(gu.run_fwd(binding, oracle, "cast", x, round=rnd), gu.run_ref(oracle, "cast", x, round=rnd),
                        f"patterns cast round={rnd}")
    # ... and normalised: rows whose RMS estimate is far from 1 in both directions
    rng = np.random.default_rng(0)
    xr = pats[rng.integers(0, pats.size, size=(512, 256))]
    xr[(xr & 0x7F80) > 0x5D00] &= 0x0FFF | 0x8000               # |x| < 2^60: squares stay inside binary32
    for kind in ("mx", "rms"):
        got = gu.run_fwd(binding, oracle, kind, xr)
        want = gu.run_ref(oracle, kind, xr)
        if kind == "mx":
            gu.assert_exact(got, want, "random-pattern rows")
        else:
            gu.assert_within_rounding_of_rho(got, want, 32, "random-pattern rows rms")


def test_degenerate_rows(binding, oracle):
    D = 256
    one = 0x3F80
    x = np.zeros((8, D), np.uint16)
    x[1, :] = 0x8000                      # all negative zeros
    x[2, 5] = one                         # one-hot
    x[3, :] = one                         # constant
    x[4, :] = 0x0001                      # smallest subnormal everywhere
    x[5, :] = 0x7F7F                      # largest finite everywhere
    x[6, ::2] = 0x0080                    # smallest normal, alternating with zero
    x[7, :32] = 0x7F00                    # one huge block, rest tiny
    x[7, 32:] = 0x0100
    for kind, exact in (("mx", True), ("cast", True), ("rms", False)):
        got = gu.run_fwd(binding, oracle, kind, x)
        want = gu.run_ref(oracle, kind, x)
        if exact:
            gu.assert_exact(got, want, f"degenerate {kind}")
        else:
            # rows 4-7 over/underflow a binary32 sum of squares: outside the baseline's stated domain
            sel = [0, 1, 2, 3]
            gu.assert_within_rounding_of_rho(tuple(a[sel] for a in got), tuple(a[sel] for a in want), 32, "degenerate rms")
    # NVFP4, all rows: for row 6 (row scale 2^-126) rho~ / scale overflows binary32 and saturates at the largest finite
    # value, so its zeros stay zeros
    gu.assert_exact(gu.run_fwd(binding, oracle, "nvfp4", x), gu.run_ref(oracle, "nvfp4", x), "degenerate nvfp4")
    for kind in ("rms_nvfp4", "cast_nvfp4", "mx4", "cast4"):
        sel = [0, 1, 2, 3] if kind == "rms_nvfp4" else list(range(8))
        got, want = gu.run_fwd(binding, oracle, kind, x[sel]), gu.run_ref(oracle, kind, x[sel])
        if kind == "rms_nvfp4":
            assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1])
        else:
            gu.assert_exact(got, want, f"degenerate {kind}")
    # constant-row closed form straight from the GPU: scale 121, code 0x72, r~ = fl32(0.4185)
    codes, scales, r = gu.run_fwd(binding, oracle, "mx", x)
    assert np.all(scales[3] == 121) and np.all(codes[3] == 0x72) and r.view(np.uint32)[3] == 0x3ED645A2


def test_subnormal_rows_with_zeros_stay_finite(binding, oracle):
    """Rows of subnormal magnitude: 1/(r~ + eps) saturates at the largest finite binary32, so zeros stay zeros."""
    x = np.zeros((6, 128), np.uint16)
    x[0, ::2] = 0x0001
    x[1, ::2] = 0x8001
    x[1, 1::2] = 0x8000
    x[2, ::2] = 0x0080
    x[3, ::3] = 0x0003
    x[4, 5] = 0x0001
    x[5, :] = 0x0002
    for kind in ("mx", "nvfp4", "mx4", "postround"):
        got, want = gu.run_fwd(binding, oracle, kind, x), gu.run_ref(oracle, kind, x)
        if kind == "postround":
            assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1])
        else:
            gu.assert_exact(got, want, f"subnormal rows {kind}")
    for block in (16, 64):
        gu.assert_exact(gu.run_fwd(binding, oracle, "mx", x, block=block), gu.run_ref(oracle, "mx", x, block=block), "subnormal rows")
    got = gu.run_fwd(binding, oracle, "rms", x)
    want = gu.run_ref(oracle, "rms", x)
    assert np.all((got[0][:, 1::2] & 0x7F)[:3] == 0) and not np.any((got[0] & 0x7F) == 0x7F)


def test_nvfp4_at_the_edge_of_the_stated_domain(binding, oracle):
    """Row scales 2^-100 and 2^+100, blocks whose E4M3 scale is subnormal or zero, global scales that push the scale
    into saturation: every byte must equal the oracle's."""
    base, _ = rows(48, 512, seed=91)
    bv = (base.astype(np.uint32) << 16).view(np.float32).copy()
    bv[:, 16:32] *= np.float32(2.0 ** -5)         # E4M3 scale in its subnormal range
    bv[:, 32:48] *= np.float32(2.0 ** -12)        # scale rounds to zero: codes +-0
    bv[:, 48:64] *= np.float32(2.0 ** -9)         # at the bottom of the subnormal range
    base = wl.f32_to_bf16_bits(bv)
    want0 = gu.run_ref(oracle, "nvfp4", base)
    assert np.any((want0[1][:, 1] > 0) & (want0[1][:, 1] < 8)) and np.all(want0[1][:, 2] == 0)
    for k in (-100, -90, 0, 90, 100):
        xs = wl.f32_to_bf16_bits(bv * np.float32(2.0 ** k))
        for p, eps in ((2, 0.0), (1, 0.0)):
            got = gu.run_fwd(binding, oracle, "nvfp4", xs, p=p, eps=eps)
            gu.assert_exact(got, gu.run_ref(oracle, "nvfp4", xs, p=p, eps=eps), f"nvfp4 row scale 2^{k}")
        if k in (-100, 100):
            assert np.array_equal(got[0], gu.run_ref(oracle, "nvfp4", base, p=1)[0])      # the shift changes no code
        gu.assert_exact(gu.run_fwd(binding, oracle, "cast_nvfp4", xs), gu.run_ref(oracle, "cast_nvfp4", xs), "mx_cast_nvfp4 at the edge")
    for gs in (2.0 ** -8, 64.0, 2.0 ** 12):        # tiny scales / scales saturating at 448
        got = gu.run_fwd(binding, oracle, "nvfp4", base, global_scale=gs)
        gu.assert_exact(got, gu.run_ref(oracle, "nvfp4", base, global_scale=gs), f"nvfp4 global scale {gs}")


@pytest.mark.parametrize("T,D", [(1, 16), (5, 48), (37, 768), (130, 1024), (33, 4096), (5, 8192), (3, 16384), (257, 2048),
                                 (7, 3072), (6, 5120), (4, 7168), (3, 10240), (3, 12288), (3, 14336), (11, 1280),
                                 (9, 2560), (131, 2560), (10, 1536), (6, 3584), (133, 1280), (131, 512), (133, 1536)])
def test_nvfp4_matches_oracle_bit_for_bit(binding, oracle, T, D):
    x, _ = rows(T, D, seed=11 * T + D)
    for p, eps, gs in ((2, 1e-5, 1.0), (1, 0.0, 1.0), (2, 0.0, 8.0)):
        got = gu.run_fwd(binding, oracle, "nvfp4", x, p=p, eps=eps, global_scale=gs)
        gu.assert_exact(got, gu.run_ref(oracle, "nvfp4", x, p=p, eps=eps, global_scale=gs), f"nvfp4 {T}x{D} p={p}")
    got = gu.run_fwd(binding, oracle, "nvfp4", x, layout=1)
    gu.assert_exact(got, gu.run_ref(oracle, "nvfp4", x), "nvfp4 tiled scales")
    # the cast without a normaliser (weights)
    for gs, layout in ((1.0, 0), (0.25, 1)):
        got = gu.run_fwd(binding, oracle, "cast_nvfp4", x, global_scale=gs, layout=layout)
        gu.assert_exact(got, gu.run_ref(oracle, "cast_nvfp4", x, global_scale=gs), f"mx_cast_nvfp4 {T}x{D} g={gs}")


@pytest.mark.parametrize("D,blocks,T", [(512, (16, 32, 64), 12288 + 5), (768, (16,), 12288 + 5), (1280, (16,), 12288 + 5),
                                        (256, (16, 32, 64), 24576 + 5)])
def test_many_short_rows_take_several_rows_per_warp(binding, oracle, D, blocks, T):
    """From about twelve thousand rows on, rows of 512, 768 (blocks of 16) and 1280 elements (blocks of 16, MXNorm statistic)
    run several to a warp, from twenty-four thousand on rows of 256 too; the odd row count leaves the last warp a partial run."""
    x, _ = rows(T, D, seed=19 + D)
    for block in blocks:
        for layout in (0, 1):
            got = gu.run_fwd(binding, oracle, "mx", x, block=block, eps=1e-5, layout=layout)
            gu.assert_exact(got, gu.run_ref(oracle, "mx", x, block=block, eps=1e-5), f"mxnorm B={block} layout={layout} {T}x{D}")
        got = gu.run_fwd(binding, oracle, "mx", x, block=block, p=1)
        gu.assert_exact(got, gu.run_ref(oracle, "mx", x, block=block, p=1), f"mxnorm p=1 B={block} {T}x{D}")
        got = gu.run_fwd(binding, oracle, "mx4", x, block=block, eps=1e-5, layout=1)
        gu.assert_exact(got, gu.run_ref(oracle, "mx4", x, block=block, eps=1e-5), f"mxnorm_mxfp4 B={block} {T}x{D}")
        if D != 1280:     # the other statistics take this kernel at D = 512 and 768 only
            got = gu.run_fwd(binding, oracle, "cast", x, block=block)
            gu.assert_exact(got, gu.run_ref(oracle, "cast", x, block=block), f"mx_cast B={block} {T}x{D}")
            got = gu.run_fwd(binding, oracle, "cast4", x, block=block)
            gu.assert_exact(got, gu.run_ref(oracle, "cast4", x, block=block), f"mx_cast_fp4 B={block} {T}x{D}")
            got = gu.run_fwd(binding, oracle, "rms", x, block=block, eps=1e-5)
            gu.assert_within_rounding_of_rho(got, gu.run_ref(oracle, "rms", x, block=block, eps=1e-5), block, "rms")
            got = gu.run_fwd(binding, oracle, "rms4", x, block=block, eps=1e-5)
            gu.assert_within_rounding_of_rho(got, gu.run_ref(oracle, "rms4", x, block=block, eps=1e-5), block, "rmsnorm_mxfp4", fp4=True)
    if D != 1280:
        got = gu.run_fwd(binding, oracle, "nvfp4", x, eps=1e-5, layout=1)
        gu.assert_exact(got, gu.run_ref(oracle, "nvfp4", x, eps=1e-5), f"nvfp4 {T}x{D}")
        got = gu.run_fwd(binding, oracle, "cast_nvfp4", x, global_scale=0.25)
        gu.assert_exact(got, gu.run_ref(oracle, "cast_nvfp4", x, global_scale=0.25), f"mx_cast_nvfp4 {T}x{D}")


def test_gain_is_applied_after_the_normaliser(binding, oracle):
    """Rows on which (x * rho~) * gamma and (x * gamma) * rho~ round to different E4M3 codes (found by search; the CPU pin of
    the oracle uses the same rows): the kernels must take the first order, for MXNorm and for the conventional path."""
    xb = np.zeros((3, 32), np.uint16)
    xb[:, 0] = wl.f32_to_bf16_bits(np.array([2.5, 2.5, 5.0], np.float32))
    xb[:, 1] = wl.f32_to_bf16_bits(np.array([-1.125, 0.28125, -0.5625], np.float32))
    gb = np.full(32, 0x3F80, np.uint16)
    gb[1] = wl.f32_to_bf16_bits(np.array([0.7265625], np.float32))[0]
    got = gu.run_fwd(binding, oracle, "mx", xb, gb)
    gu.assert_exact(got, gu.run_ref(oracle, "mx", xb, gb), "gain order")
    assert list(got[0][:, 1]) == [229, 85, 213]


def test_power_of_two_shift_on_gpu(binding, oracle):
    x, _ = rows(64, 1024, seed=23)
    xv = (x.astype(np.uint32) << 16).view(np.float32)
    base = gu.run_fwd(binding, oracle, "mx", x)
    for k in (-9, 4):
        xs = wl.f32_to_bf16_bits(xv * np.float32(2.0 ** k))
        c, s, r = gu.run_fwd(binding, oracle, "mx", xs)
        assert np.array_equal(c, base[0]) and np.array_equal(s, base[1])
        assert np.array_equal(r, base[2] * np.float32(2.0 ** k))


def test_runs_are_bitwise_repeatable(binding, oracle):
    x, gain = rows(300, 4096, seed=29)
    for kind in ("mx", "rms", "nvfp4"):
        a = gu.run_fwd(binding, oracle, kind, x, eps=1e-5)
        b = gu.run_fwd(binding, oracle, kind, x, eps=1e-5)
        assert all(np.array_equal(u, v) for u, v in zip(a, b))


def test_rms_output_is_optional_and_stream_is_honoured(binding, oracle):
    x_bits, _ = rows(64, 1024, seed=31)
    x = wl.from_bits(x_bits).cuda()
    codes, scales, rms = binding.alloc_outputs(64, 1024)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        binding.mxnorm_fwd(x, None, codes, scales, None, eps=1e-5, stream=s)
    s.synchronize()
    want = gu.run_ref(oracle, "mx", x_bits, eps=1e-5)
    assert np.array_equal(codes.cpu().numpy(), want[0]) and np.array_equal(scales.cpu().numpy().reshape(64, 32), want[1])


@pytest.mark.parametrize("block", [16, 32, 64])
@pytest.mark.parametrize("T,D", [(1, 64), (37, 768), (130, 1024), (33, 4096), (9, 2560), (5, 8192), (3, 16384), (257, 2048), (133, 1280),
                                 (7, 3072), (6, 5120), (5, 6144), (4, 7168), (3, 10240), (3, 12288), (3, 14336), (10, 1536), (6, 3584), (131, 512), (7, 512)])
def test_mxfp4_matches_oracle(binding, oracle, T, D, block):
    """E2M1 codes with E8M0 scales (the paper's cast with the element type set to E2M1)."""
    x, _ = rows(T, D, seed=13 * T + D + block)
    for p, eps in ((2, 1e-5), (1, 0.0)):
        got = gu.run_fwd(binding, oracle, "mx4", x, block=block, p=p, eps=eps)
        gu.assert_exact(got, gu.run_ref(oracle, "mx4", x, block=block, p=p, eps=eps), f"mxnorm_mxfp4 B={block} p={p} {T}x{D}")
    got = gu.run_fwd(binding, oracle, "cast4", x, block=block)
    gu.assert_exact(got, gu.run_ref(oracle, "cast4", x, block=block), f"mx_cast_fp4 B={block}")
    got = gu.run_fwd(binding, oracle, "rms4", x, block=block, eps=1e-5)
    gu.assert_within_rounding_of_rho(got, gu.run_ref(oracle, "rms4", x, block=block, eps=1e-5), block, "rmsnorm_mxfp4", fp4=True)
    got = gu.run_fwd(binding, oracle, "mx4", x, block=block, eps=1e-5, layout=1)
    gu.assert_exact(got, gu.run_ref(oracle, "mx4", x, block=block, eps=1e-5), "mxnorm_mxfp4 tiled scales")


def test_mxfp4_degenerate_rows_and_patterns(binding, oracle):
    pats = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    pats = pats[(pats & 0x7F80) != 0x7F80]
    x = np.zeros((pats.size, 32), np.uint16)
    x[:, 0] = pats
    x[:, 17] = (pats >> 1) & 0x7FFF
    x[(x[:, 17] & 0x7F80) == 0x7F80, 17] = 0
    gu.assert_exact(gu.run_fwd(binding, oracle, "cast4", x), gu.run_ref(oracle, "cast4", x), "fp4 patterns")
    z = np.zeros((4, 128), np.uint16)
    z[1, :] = 0x8000
    z[2, 7] = 0x3F80
    z[3, :] = 0x3F80
    codes, scales, r = gu.run_fwd(binding, oracle, "mx4", z)
    gu.assert_exact((codes, scales, r), gu.run_ref(oracle, "mx4", z), "fp4 degenerate")
    assert np.all(scales[3] == 127) and np.all(codes[3] == 0x44)      # constant row closed form


@pytest.mark.parametrize("T,D", [(5, 48), (37, 768), (33, 4096), (6, 5120), (3, 16384), (257, 2048)])
def test_rmsnorm_nvfp4_matches_oracle(binding, oracle, T, D):
    """The conventional path in NVFP4: r within 1e-6, E4M3 scale bytes and E2M1 codes within the rounding of rho."""
    x, _ = rows(T, D, seed=17 * T + D)
    for eps, gs in ((1e-5, 1.0), (0.0, 4.0)):
        gc, gs_, gr = gu.run_fwd(binding, oracle, "rms_nvfp4", x, eps=eps, global_scale=gs)
        wc, ws, wr = gu.run_ref(oracle, "rms_nvfp4", x, eps=eps, global_scale=gs)
        assert np.all(np.abs(gr.astype(np.float64) - wr) <= 1e-6 * np.abs(wr))
        sdiff = gs_ != ws                                   # an E4M3 scale can move by one code when rho rounds differently
        assert sdiff.mean() <= 1e-4 and np.all(np.abs(gs_.astype(int) - ws.astype(int)) <= 1)
        keep = ~np.repeat(sdiff, 16, axis=1)
        d = gu.nibble_steps(gc, wc)[keep]
        assert d.max(initial=0) <= 1 and (d != 0).mean() <= 1e-4


def test_division_shortcuts_equal_ieee_division(binding):
    assert binding.selftest_division() == 0


@pytest.mark.parametrize("block", [16, 32, 64])
@pytest.mark.parametrize("T,D", [(5, 64), (37, 768), (33, 4096), (9, 2560), (3, 16384), (257, 2048)])
def test_postround_mxnorm_matches_oracle(binding, oracle, T, D, block):
    """The paper's ablation: RMS from power-of-two-rounded absmaxes through the f^-1 table.  The library and the oracle
    each build their own table, so r~ is compared to 1e-6 and scales/codes within the rounding of rho."""
    x, _ = rows(T, D, seed=19 * T + D + block)
    x[0] = 0                                                    # a zero row
    for eps in (1e-5, 0.0):
        got = gu.run_fwd(binding, oracle, "postround", x, block=block, eps=eps)
        want = gu.run_ref(oracle, "postround", x, block=block, eps=eps)
        nz = want[2] != 0
        assert np.all(got[2][~nz] == 0)
        sel = lambda t: tuple(a[nz] for a in t)
        gu.assert_within_rounding_of_rho(sel(got), sel(want), block, f"postround B={block} {T}x{D}")
        assert np.array_equal(got[0][~nz], want[0][~nz]) and np.array_equal(got[1][~nz], want[1][~nz])
    got = gu.run_fwd(binding, oracle, "postround", x, block=block, eps=1e-5, layout=1)
    want = gu.run_ref(oracle, "postround", x, block=block, eps=1e-5)
    nz = want[2] != 0
    gu.assert_within_rounding_of_rho(tuple(a[nz] for a in got), tuple(a[nz] for a in want), block, "postround tiled")


@pytest.mark.parametrize("block", [16, 32, 64])
@pytest.mark.parametrize("T,D", [(5, 64), (37, 768), (33, 4096), (9, 2560), (3, 16384), (257, 2048)])
def test_residual_add_then_mxnorm_matches_oracle(binding, oracle, T, D, block):
    x, _ = rows(T, D, seed=23 * T + D + block)
    res, _ = rows(T, D, seed=29 * T + D + block)
    res[0] = x[0] ^ 0x8000                                      # exact cancellation: a zero row
    want_h, wc, ws, wr = oracle.mxnorm_add_ref(x, res, eps=1e-5, block=block)
    xg, rg = wl.from_bits(x).cuda(), wl.from_bits(res).cuda()
    for inplace in (False, True):
        hfull, hbytes = gu.guarded(T * D * 2)
        h = hbytes.view(torch.bfloat16).view(T, D)
        codes, scales, rms = binding.alloc_outputs(T, D, block)
        target = xg.clone() if inplace else h
        binding.mxnorm_add_fwd(target if inplace else xg, rg, target, codes, scales, rms, eps=1e-5, block=block)
        torch.cuda.synchronize()
        assert gu.guards_intact(hfull, T * D * 2)
        assert np.array_equal(wl.bits(target.cpu()), want_h)
        assert np.array_equal(codes.cpu().numpy(), wc)
        assert np.array_equal(scales.cpu().numpy().reshape(T, D // block), ws)
        assert np.array_equal(rms.cpu().numpy(), wr)
