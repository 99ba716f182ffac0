"""Pins for the CPU oracle: values the paper prints, closed forms, invariants, brute force on
tiny inputs and library special cases.  None of these tests touches the GPU path."""
import math
import os

import numpy as np
import pytest
import torch

from paper_2603_13180_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

ONE = 0x3F80  # bf16 1.0


def _read_table(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def bf16_bits(a):
    return wl.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def bf16_vals(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32)


# ------------------------------------------------------------------ brute-force definitions
E4M3_POS = np.array([(m * 2.0 ** -9) if e == 0 else (8 + m) * 2.0 ** (e - 10)
                     for e in range(16) for m in range(8)][:127], dtype=np.float64)  # codes 0..0x7E
E2M1_POS = np.array([0, .5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)


def nearest_code(q, grid):
    """Definition of round-to-nearest, ties to the even code, saturating: search the whole grid."""
    q = np.asarray(q, dtype=np.float64)
    a = np.abs(q)[..., None]
    diff = np.abs(a - grid)                       # [..., G]
    best = diff.min(axis=-1, keepdims=True)
    cand = diff == best                           # one or two candidates
    idx = np.arange(grid.size)
    even_first = np.where(cand & (idx % 2 == 0), idx, np.where(cand, idx + 1000, 10 ** 6))
    code = even_first.min(axis=-1) % 1000
    return code.astype(np.uint8), np.signbit(q)


def smallest_pow2_scale(m, emax=8):
    """Definition of the paper's scale: smallest S = 2^(sb-127), sb in [0,254], with m/S <= 2^emax
    (zero block -> sb 0)."""
    m = np.asarray(m, dtype=np.float64)
    sb = np.arange(255)
    S = np.ldexp(1.0, sb - 127)
    ok = (m[..., None] / S) <= 2.0 ** emax
    first = np.where(ok, sb, 10 ** 6).min(axis=-1)
    first = np.where(first == 10 ** 6, 254, first)
    return np.where(m == 0, 0, first).astype(np.uint8)


# ------------------------------------------------------------------ P1: the constants
def closed_form_coef(B, p):
    """RMS/G_p for i.i.d. standard normal blocks: E[max_b |Z_b|^p] = int_0^inf p x^(p-1) P(max > x) dx."""
    from scipy import integrate, special
    f = lambda x: p * x ** (p - 1) * (1.0 - special.erf(x / math.sqrt(2.0)) ** B)
    val, _ = integrate.quad(f, 0, 12, epsabs=1e-13, epsrel=1e-13, limit=400)
    return val ** (-1.0 / p)


def test_constants_match_closed_form_and_printed_table(oracle):
    for B, p, c in _read_table("absmax_scale_factor.txt"):
        B, p, c = int(B), int(p), float(c)
        assert abs(closed_form_coef(B, p) - c) < 1.0e-4, (B, p)   # Monte-Carlo constant, 4 printed digits
        assert oracle.coef(B, p) == np.float32(c)                  # the oracle holds the printed value
        assert c < 1.0                                             # direction: RMS/G, not G/RMS


def test_constant_direction_monte_carlo(oracle):
    # Theorem 1: G_p / RMS -> 1/coef, so coef * G_p estimates the RMS of Gaussian rows.
    rng = np.random.default_rng(0)
    for B, p in ((16, 2), (32, 2), (32, 1), (64, 2)):
        z = rng.standard_normal((4000, 64 * B))
        m = np.abs(z.reshape(4000, 64, B)).max(-1)
        G = (m ** p).mean(-1) ** (1.0 / p)
        rms = np.sqrt((z ** 2).mean(-1))
        assert abs((oracle.coef(B, p) * G / rms).mean() - 1.0) < 3e-3


# ------------------------------------------------------------------ P2: printed worked values
def test_printed_output_bounds_on_one_hot_rows(oracle):
    for norm, p, D, B, bound in _read_table("output_bounds.txt"):
        p, D, B, bound = int(p), int(D), int(B), float(bound)
        x = np.zeros((1, D), np.uint16)
        x[0, 37] = bf16_bits([3.0])[0]
        if norm == "mxnorm":
            codes, scales, r = oracle.mxnorm_ref(x, p=p, block=B)
        else:
            codes, scales, r = oracle.rmsnorm_mxfp8_ref(x, block=B)
        normalised = 3.0 / float(r[0])
        assert abs(normalised - bound) < 0.006, (norm, p, normalised)   # printed to 2 decimals
        # the emitted MX tensor dequantises to the same value within E4M3 precision (2^-4 relative)
        k = 37 // B
        deq = oracle.e4m3_decode(int(codes[0, 37])) * 2.0 ** (int(scales[0, k]) - 127)
        assert abs(deq - normalised) <= normalised * 2.0 ** -4
        assert np.all(np.delete(codes[0], 37) == 0) and np.all(np.delete(scales[0], k) == 0)


def test_lemma_bounds_hold_on_random_rows(oracle):
    x = wl.bits(wl.gaussian(64, 1024, seed=3, row_scale_sigma=1.0))
    xv = bf16_vals(x).astype(np.float64)
    for B, p in ((16, 1), (16, 2), (32, 2)):
        _, _, r = oracle.mxnorm_ref(x, p=p, block=B)
        K = 1024 // B
        assert np.all(np.abs(xv).max(-1) / r <= K ** (1.0 / p) / oracle.coef(B, p) * (1 + 1e-6))
    _, _, r = oracle.rmsnorm_mxfp8_ref(x)
    assert np.all(np.abs(xv).max(-1) / r <= math.sqrt(1024) * (1 + 1e-6))


# ------------------------------------------------------------------ P4: constant row closed form
@pytest.mark.parametrize("a", [1.0, -1.0, 0.007, 3.0e4])
def test_constant_row_closed_form(oracle, a):
    ab = bf16_bits([a])[0]
    av = float(bf16_vals(np.array([ab], np.uint16))[0])
    x = np.full((3, 256), ab, np.uint16)
    codes, scales, r = oracle.mxnorm_ref(x, p=2, block=32)
    # every block absmax is |a| -> G = |a| -> r~ = fl32(0.4185 * |a|); x*rho~ = +-1/0.4185 = +-2.389..
    assert np.all(r == np.float32(np.float64(np.float32(0.4185)) * abs(av)))
    # 2.389 lies in (2,4]: S = 2^(2-8) -> biased 121; q = 2.389*64 = 152.9 -> nearest E4M3 is 160 = 0x72
    assert np.all(scales == 121)
    assert np.all(codes == (0x72 if av > 0 else 0xF2))
    if a == 1.0:
        assert r.view(np.uint32)[0] == 0x3ED645A2
    # OCP floor rounding puts the scale one binade lower and the code at 2.389*128 = 305.9 -> 320 = 0x7A
    codes_f, scales_f, _ = oracle.mxnorm_ref(x, p=2, block=32, mode=oracle.ROUND_FLOOR_OCP)
    assert np.all(scales_f == 120) and np.all((codes_f & 0x7F) == 0x7A)
    # p = 1 and B = 16: same structure with the other constants
    _, _, r1 = oracle.mxnorm_ref(x, p=1, block=16)
    assert np.all(r1 == np.float32(np.float64(np.float32(0.4814)) * abs(av)))


def test_epsilon_enters_the_denominator(oracle):
    # rho~ = 1 / (r~ + eps): with a constant row of ones and eps = 0.5, r~ = 0.4185 and x*rho~ = 1/0.9185 = 1.0887,
    # which lies in (1,2]: S = 2^(1-8) (biased 120), q = 1.0887*128 = 139.4 -> nearest E4M3 value 144 = 0x71;
    # r~ itself is reported without eps
    x = np.full((2, 128), ONE, np.uint16)
    codes, scales, r = oracle.mxnorm_ref(x, eps=0.5)
    assert np.all(r == np.float32(0.4185)) and np.all(scales == 120) and np.all(codes == 0x71)
    codes, scales, r = oracle.mxnorm_nvfp4_ref(x, eps=0.5)
    # B = 16: x*rho~ = 1/0.9688 = 1.0322; scale = E4M3(1.0322/6 = 0.17203) = 0.171875 = 0x23; q = 6.0055 -> 6 -> 0x77
    assert np.all(r == np.float32(0.4688)) and np.all(scales == 0x23) and np.all(codes == 0x77)
    # a zero row stays zero whatever eps is
    z = np.zeros((1, 64), np.uint16)
    codes, scales, r = oracle.mxnorm_ref(z, eps=0.5)
    assert np.all(codes == 0) and np.all(scales == 0) and np.all(r == 0)


def test_nvfp4_constant_row_closed_form(oracle):
    x = np.full((2, 64), ONE, np.uint16)
    codes, scales, r = oracle.mxnorm_nvfp4_ref(x)
    assert np.all(r == np.float32(0.4688))
    # x*rho~ = 2.1331; block scale = nearest E4M3 to 2.1331/6 = 0.35552 -> 0.34375 = 0x2B;
    # q = 2.1331/0.34375 = 6.205 -> saturates at 6 -> nibble 7, two per byte -> 0x77
    assert np.all(scales == 0x2B)
    assert np.all(codes == 0x77)
    xn = np.full((2, 64), ONE | 0x8000, np.uint16)
    codes_n, scales_n, _ = oracle.mxnorm_nvfp4_ref(xn)
    assert np.all(scales_n == 0x2B) and np.all(codes_n == 0xFF)


def test_zero_rows(oracle):
    x = np.zeros((2, 128), np.uint16)
    x[1, ::2] = 0x8000  # negative zeros
    for fn in (lambda: oracle.mxnorm_ref(x), lambda: oracle.rmsnorm_mxfp8_ref(x)):
        codes, scales, r = fn()
        assert np.all(r == 0) and np.all(scales == 0)
        assert np.all(codes[0] == 0) and np.all(codes[1, ::2] == 0x80) and np.all(codes[1, 1::2] == 0)
    codes, scales = oracle.mx_cast_ref(x)
    assert np.all(scales == 0) and np.all(codes[1, ::2] == 0x80)
    codes, scales, r = oracle.mxnorm_nvfp4_ref(x)
    assert np.all(r == 0) and np.all(scales == 0) and np.all(codes[0] == 0) and np.all(codes[1] == 0x08)


# ------------------------------------------------------------------ P3: invariants
def _rand_rows(seed, T=48, D=512, sigma=1.5):
    return wl.bits(wl.gaussian(T, D, seed=seed, row_scale_sigma=sigma))


@pytest.mark.parametrize("k", [-20, -3, 1, 7, 30])
def test_power_of_two_shift_invariance(oracle, k):
    x = _rand_rows(1)
    xs = bf16_bits(bf16_vals(x) * np.float32(2.0 ** k))  # exact in bf16 (no subnormals at these sizes)
    assert np.array_equal(bf16_vals(xs), bf16_vals(x) * np.float32(2.0 ** k))
    c0, s0 = oracle.mx_cast_ref(x)
    c1, s1 = oracle.mx_cast_ref(xs)
    assert np.array_equal(c0, c1) and np.array_equal(s1.astype(int), s0.astype(int) + k)
    for p, B in ((2, 32), (1, 32), (2, 16), (2, 64)):
        c0, s0, r0 = oracle.mxnorm_ref(x, p=p, block=B)
        c1, s1, r1 = oracle.mxnorm_ref(xs, p=p, block=B)
        assert np.array_equal(c0, c1) and np.array_equal(s0, s1)
        assert np.array_equal(r1, r0 * np.float32(2.0 ** k))
    c0, s0, r0 = oracle.mxnorm_nvfp4_ref(x)
    c1, s1, r1 = oracle.mxnorm_nvfp4_ref(xs)
    assert np.array_equal(c0, c1) and np.array_equal(s0, s1) and np.array_equal(r1, r0 * np.float32(2.0 ** k))
    c0, s0, r0 = oracle.rmsnorm_mxfp8_ref(x)
    c1, s1, r1 = oracle.rmsnorm_mxfp8_ref(xs)
    assert np.array_equal(c0, c1) and np.array_equal(s0, s1)


def test_block_permutation_and_negation(oracle):
    x = _rand_rows(2, T=16, D=512)
    perm = np.random.default_rng(0).permutation(16)
    xp = x.reshape(16, 16, 32)[:, perm, :].reshape(16, 512)
    c0, s0, r0 = oracle.mxnorm_ref(x)
    c1, s1, r1 = oracle.mxnorm_ref(xp)
    assert np.array_equal(r0, r1)
    assert np.array_equal(c0.reshape(16, 16, 32)[:, perm, :].reshape(16, 512), c1)
    assert np.array_equal(s0[:, perm], s1)
    cn, sn, rn = oracle.mxnorm_ref(x ^ 0x8000)
    assert np.array_equal(cn, c0 ^ 0x80) and np.array_equal(sn, s0) and np.array_equal(rn, r0)


def test_default_rounding_uses_top_binade(oracle):
    x = _rand_rows(4)
    for codes, scales in (oracle.mx_cast_ref(x), oracle.mxnorm_ref(x)[:2], oracle.rmsnorm_mxfp8_ref(x)[:2]):
        blockmax = (codes & 0x7F).reshape(codes.shape[0], -1, 32).max(-1)
        # max |q| per non-zero block lies in (128, 256]: E4M3 codes 0x71..0x78 (0x70 = 128 only by rounding down from <136)
        assert np.all((blockmax >= 0x70) & (blockmax <= 0x78))


# ------------------------------------------------------------------ P6: brute force
def test_all_bf16_patterns_against_definitions(oracle):
    pats = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    finite = (pats & 0x7F80) != 0x7F80
    pats = pats[finite]
    x = np.zeros((pats.size, 32), np.uint16)
    x[:, 0] = pats                       # block absmax = |pattern|
    x[:, 1] = pats >> 1                  # a second, smaller element with other mantissa bits
    x[:, 1] &= 0x7FFF
    x[(x[:, 1] & 0x7F80) == 0x7F80, 1] = 0
    xv = bf16_vals(x).astype(np.float64)
    m = np.abs(xv).max(-1)
    codes, scales = oracle.mx_cast_ref(x)
    sb = smallest_pow2_scale(m)
    assert np.array_equal(scales[:, 0], sb)
    S = np.ldexp(1.0, sb.astype(int) - 127)
    for col in (0, 1):
        code, neg = nearest_code(xv[:, col] / S, E4M3_POS)
        assert np.array_equal(codes[:, col], code | (neg.astype(np.uint8) << 7)), col
    # floor (OCP) mode: scale exponent = floor(log2 m) - 8, codes saturate at 448
    codes_f, scales_f = oracle.mx_cast_ref(x, mode=oracle.ROUND_FLOOR_OCP)
    nz = m > 0
    fl = np.floor(np.log2(m[nz])).astype(int)      # log2 of a bf16 value: exact enough for floor (8-bit significand)
    frac, ex = np.frexp(m[nz])
    assert np.array_equal(fl, ex - 1)
    assert np.array_equal(scales_f[nz, 0].astype(int), np.clip(ex - 1 - 8 + 127, 0, 254))
    Sf = np.ldexp(1.0, scales_f[:, 0].astype(int) - 127)
    code, neg = nearest_code(xv[:, 0] / Sf, E4M3_POS)
    assert np.array_equal(codes_f[:, 0], code | (neg.astype(np.uint8) << 7))
    # RCEIL on max (divide by 448): smallest power of two >= fl32(m/448)
    codes_m, scales_m = oracle.mx_cast_ref(x, mode=oracle.ROUND_RCEIL_MAX)
    t = (m.astype(np.float32) / np.float32(448.0)).astype(np.float64)
    sbm = np.arange(255)
    ok = np.ldexp(1.0, sbm - 127) >= t[:, None]
    want = np.where(t == 0, 0, np.where(ok, sbm, 10 ** 6).min(-1))
    assert np.array_equal(scales_m[:, 0].astype(int), want)


def test_e4m3_encoder_exhaustive_neighbourhoods(oracle):
    # every code value, every midpoint between neighbours, and values just off the midpoints
    g = E4M3_POS
    mids = (g[:-1] + g[1:]) / 2
    probes = np.concatenate([g, mids, np.nextafter(mids.astype(np.float32), np.float32(0)),
                             np.nextafter(mids.astype(np.float32), np.float32(1e9)),
                             [448.0, 463.9, 464.0, 465.0, 480.0, 1e6, 2.0 ** -10, 2.0 ** -10 * 1.001,
                              2.0 ** -11, 1e-30]])
    probes = probes.astype(np.float32)
    want, _ = nearest_code(probes.astype(np.float64), g)
    got = np.array([oracle.e4m3_encode(float(v)) for v in probes], np.uint8)
    assert np.array_equal(got, want)
    gotn = np.array([oracle.e4m3_encode(float(-v)) for v in probes], np.uint8)
    assert np.array_equal(gotn, want | 0x80)
    for c in range(127):
        assert oracle.e4m3_decode(c) == g[c] and oracle.e4m3_decode(c | 0x80) == -g[c]
    assert oracle.e4m3_encode(float("nan")) & 0x7F == 0x7F
    assert oracle.e4m3_encode(3e38) == 0x7E and oracle.e4m3_encode(float("-inf")) == 0xFE   # saturating


def test_e2m1_encoder_exhaustive_neighbourhoods(oracle):
    g = E2M1_POS
    mids = (g[:-1] + g[1:]) / 2        # 0.25 .75 1.25 1.75 2.5 3.5 5
    probes = np.concatenate([g, mids, np.nextafter(mids.astype(np.float32), np.float32(0)),
                             np.nextafter(mids.astype(np.float32), np.float32(1e9)), [6.5, 7.0, 100.0, 1e-20]])
    probes = probes.astype(np.float32)
    want, _ = nearest_code(probes.astype(np.float64), g)
    got = np.array([oracle.e2m1_encode(float(v)) for v in probes], np.uint8)
    assert np.array_equal(got, want)
    # the ties listed for RN-even on this grid
    for v, c in ((0.25, 0), (0.75, 2), (1.25, 2), (1.75, 4), (2.5, 4), (3.5, 6), (5.0, 6)):
        assert oracle.e2m1_encode(v) == c and oracle.e2m1_encode(-v) == (c | 8)


def test_mxnorm_scales_and_codes_by_definition_given_rho(oracle):
    """Given the emitted r~ (pinned elsewhere), scales and codes must be the definitional
    smallest-power-of-two scale of fl32(m*rho~) and the nearest E4M3 value of fl32(x*rho~)/S."""
    x = wl.bits(wl.make_inputs(wl.Workload("t", 24, 768, seed=5, outlier_frac=0.004))["x"])
    xv = bf16_vals(x)
    for eps in (0.0, 1e-5):
        for B in (16, 32, 64):
            codes, scales, r = oracle.mxnorm_ref(x, eps=eps, block=B)
            rho = (np.float32(1.0) / (r + np.float32(eps))).astype(np.float32)
            y = (xv * rho[:, None]).astype(np.float32)            # fl32(x * rho~)
            m = np.abs(y).reshape(24, -1, B).max(-1)
            sb = smallest_pow2_scale(m)
            assert np.array_equal(scales, sb)
            S = np.repeat(np.ldexp(1.0, sb.astype(int) - 127), B, axis=1)
            code, neg = nearest_code(y.astype(np.float64) / S, E4M3_POS)
            assert np.array_equal(codes, code | (neg.astype(np.uint8) << 7))
    # the same tail with the true RMS and a gain (Algorithm 1)
    gain = bf16_bits(1.0 + 0.1 * np.random.default_rng(1).standard_normal(768))
    codes, scales, r = oracle.rmsnorm_mxfp8_ref(x, gain=gain, eps=1e-5)
    rho = (np.float32(1.0) / r).astype(np.float32)
    y = ((xv * rho[:, None]).astype(np.float32) * bf16_vals(gain)[None, :]).astype(np.float32)
    m = np.abs(y).reshape(24, -1, 32).max(-1)
    sb = smallest_pow2_scale(m)
    assert np.array_equal(scales, sb)
    code, neg = nearest_code(y.astype(np.float64) / np.repeat(np.ldexp(1.0, sb.astype(int) - 127), 32, axis=1), E4M3_POS)
    assert np.array_equal(codes, code | (neg.astype(np.uint8) << 7))


def test_mxnorm_with_gain_by_definition_and_closed_forms(oracle):
    """The gain extension of Algorithm 2 (the paper folds the gain into the next weight, Sec. 3.7): rho~ is estimated
    from |x| alone, then scales and codes come from y = fl32(fl32(x * rho~) * gamma).  Estimating rho~ from x * gamma,
    or multiplying by gamma before rho~, fails one of the checks below."""
    x = wl.bits(wl.make_inputs(wl.Workload("t", 24, 768, seed=15, outlier_frac=0.004))["x"])
    xv = bf16_vals(x)
    gain = bf16_bits(1.0 + 0.3 * np.random.default_rng(4).standard_normal(768))
    gv = bf16_vals(gain)
    for B, p, eps in ((32, 2, 1e-5), (16, 1, 0.0), (64, 2, 0.0)):
        codes, scales, r = oracle.mxnorm_ref(x, gain=gain, p=p, eps=eps, block=B)
        # r~ does not see the gain: same bits as without it, and equal to coef * G_p(|x|) recomputed here
        assert np.array_equal(r, oracle.mxnorm_ref(x, p=p, eps=eps, block=B)[2])
        m = np.abs(xv.astype(np.float64)).reshape(24, -1, B).max(-1)
        want_r = np.float64(np.float32(oracle.coef(B, p))) * (m ** p).mean(-1) ** (1.0 / p)
        assert np.all(np.abs(r - want_r) <= want_r * 2.0 ** -23)
        rho = (np.float32(1.0) / (r + np.float32(eps))).astype(np.float32)
        y = ((xv * rho[:, None]).astype(np.float32) * gv[None, :]).astype(np.float32)     # two binary32 roundings, in this order
        sb = smallest_pow2_scale(np.abs(y).reshape(24, -1, B).max(-1))
        assert np.array_equal(scales, sb)
        S = np.repeat(np.ldexp(1.0, sb.astype(int) - 127), B, axis=1)
        code, neg = nearest_code(y.astype(np.float64) / S, E4M3_POS)
        assert np.array_equal(codes, code | (neg.astype(np.uint8) << 7))
        # the other order of the two products rounds differently somewhere on these rows (the check above is not vacuous)
        y_other = (xv * (rho[:, None] * gv[None, :]).astype(np.float32)).astype(np.float32)
        assert np.any(y_other != y)
    # The order of the two products.  The last-bit difference between (x * rho~) * gamma and (x * gamma) * rho~ reaches an
    # E4M3 rounding boundary only about once in a million elements, so it is pinned on rows found by search: one block per
    # row, element 0 dominant (it fixes r~ = 0.4185 |x0| and the scale), element 1 the probe, gamma = 0.7265625 on column 1.
    xb = np.zeros((3, 32), np.uint16)
    xb[:, 0] = bf16_bits([2.5, 2.5, 5.0])
    xb[:, 1] = bf16_bits([-1.125, 0.28125, -0.5625])
    gb = np.full(32, ONE, np.uint16)
    gb[1] = bf16_bits([0.7265625])[0]
    xw, gw = bf16_vals(xb), bf16_vals(gb)
    codes, scales, r = oracle.mxnorm_ref(xb, gain=gb)
    assert np.array_equal(r, (np.float64(np.float32(0.4185)) * np.array([2.5, 2.5, 5.0])).astype(np.float32))
    rho = (np.float32(1.0) / r).astype(np.float32)

    def by_definition(y):
        sb = smallest_pow2_scale(np.abs(y).max(-1, keepdims=True))
        code, neg = nearest_code(y.astype(np.float64) / np.ldexp(1.0, sb.astype(int) - 127), E4M3_POS)
        return sb, code | (neg.astype(np.uint8) << 7)

    s_paper, c_paper = by_definition(((xw * rho[:, None]).astype(np.float32) * gw[None, :]).astype(np.float32))
    s_other, c_other = by_definition(((xw * gw[None, :]).astype(np.float32) * rho[:, None]).astype(np.float32))
    assert np.all(c_paper[:, 1] != c_other[:, 1]) and np.array_equal(s_paper, s_other)      # the orders differ on every probe
    assert np.array_equal(scales, s_paper) and np.array_equal(codes, c_paper)
    assert list(codes[:, 1]) == [229, 85, 213]
    # constant row, gamma = 2 everywhere: r~ unchanged, y doubles exactly -> every scale byte + 1, codes unchanged
    ones = np.full((2, 256), ONE, np.uint16)
    c0, s0, r0 = oracle.mxnorm_ref(ones)
    c2, s2, r2 = oracle.mxnorm_ref(ones, gain=np.full(256, 0x4000, np.uint16))
    assert np.array_equal(r2, r0) and np.all(s0 == 121) and np.all(s2 == 122) and np.array_equal(c2, c0) and np.all(c2 == 0x72)
    # one channel's gamma = 0: that element's code is 0, r~ and every other block are untouched (an estimator fed with
    # x * gamma would see a smaller block maximum in block 0 of a one-hot-dominated row and change r~)
    xo = np.full((1, 128), ONE, np.uint16)
    xo[0, 5] = bf16_bits([100.0])[0]
    g0 = np.full(128, ONE, np.uint16)
    g0[5] = 0
    c1, s1, r1 = oracle.mxnorm_ref(xo)
    cz, sz, rz = oracle.mxnorm_ref(xo, gain=g0)
    assert np.array_equal(rz, r1) and cz[0, 5] == 0
    assert np.array_equal(cz[0, 32:], c1[0, 32:]) and np.array_equal(sz[0, 1:], s1[0, 1:])
    # block 0 now holds ones only (times rho~): its scale is the one the other all-ones blocks have
    assert sz[0, 0] == s1[0, 1] and np.all(np.delete(cz[0, :32], 5) == c1[0, 32])


def test_reciprocals_saturate_instead_of_overflowing(oracle):
    """Rows of subnormal magnitude: 1/(r~ + eps) would overflow binary32; it saturates at the largest finite binary32, so
    zeros stay zeros (no 0 * inf = NaN) and every output is the definitional cast of x * FLT_MAX."""
    FMAX = np.float32(np.finfo(np.float32).max)
    x = np.zeros((3, 64), np.uint16)
    x[0, ::2] = 0x0001                     # smallest bf16 subnormal (2^-133) alternating with zero
    x[1, ::2] = 0x8001
    x[1, 1::2] = 0x8000                    # negative values and negative zeros
    x[2, ::2] = 0x0080                     # smallest normal (2^-126) alternating with zero: rho~ ~ 2^127, still finite
    xv = bf16_vals(x)
    codes, scales, r = oracle.mxnorm_ref(x)
    assert np.all(r[:2] > 0) and np.all(r[:2] < 2.0 ** -128)            # 1/r~ overflows for rows 0 and 1
    rho = np.array([FMAX, FMAX, np.float32(1.0) / r[2]], np.float32)
    y = (xv * rho[:, None]).astype(np.float32)
    assert np.all(np.isfinite(y))
    sb = smallest_pow2_scale(np.abs(y).reshape(3, -1, 32).max(-1))
    assert np.array_equal(scales, sb)
    code, neg = nearest_code(y.astype(np.float64) / np.repeat(np.ldexp(1.0, sb.astype(int) - 127), 32, axis=1), E4M3_POS)
    assert np.array_equal(codes, code | (neg.astype(np.uint8) << 7))
    assert np.all(codes[0, 1::2] == 0) and np.all(codes[1, 1::2] == 0x80) and np.all(codes[2, 1::2] == 0)
    # the baseline's rho = 1/r and the column-wise cast's rho = 1/(r + eps) saturate the same way
    c, s, rr = oracle.rmsnorm_mxfp8_ref(x[:2])
    assert np.all((c[:, 1::2] & 0x7F) == 0) and np.all((c[:, ::2] & 0x7F) != 0x7F)
    xt = np.zeros((32, 4), np.uint16)
    xt[::2, 0] = 0x0001
    ct, st = oracle.mx_cast_transposed_ref(xt, rms=np.full(32, 2.0 ** -140, np.float32))
    assert np.all(ct[0, 1::2] == 0) and np.all(ct[0, ::2] == ct[0, 0]) and (ct[0, 0] & 0x7F) not in (0, 0x7F)
    # NVFP4: the per-block factor rho~ * g / scale saturates too.  Row 2: a = 2^-126 * rho~ = 2.133, scale 0x2B = 0.34375,
    # rho~ / 0.34375 ~ 2^128.6 overflows -> FLT_MAX; x * FLT_MAX = 4 -> nibble 6; zeros stay zeros
    c4, s4, r4 = oracle.mxnorm_nvfp4_ref(x)
    assert np.all(s4[2] == 0x2B) and np.all(c4[2] == 0x06)
    assert np.all(c4[0] & 0xF0 == 0) and np.all(c4[1] & 0xF0 == 0x80)
    # rows 0, 1: rho~ = FLT_MAX, a = 2^-133 * FLT_MAX = 2^-5 (just below): scale = E4M3(a / 6) and codes by definition
    a = (np.abs(xv[:2]).reshape(2, -1, 16).max(-1) * FMAX).astype(np.float32)
    sc, _ = nearest_code(((a / np.float32(6.0)).astype(np.float32)).astype(np.float64), E4M3_POS)
    assert np.array_equal(s4[:2], sc)
    d = E4M3_POS[sc].astype(np.float32)
    with np.errstate(over="ignore"):
        inv = np.minimum(FMAX / d, FMAX).astype(np.float32)
    q = (xv[:2] * np.repeat(inv, 16, axis=1)).astype(np.float32)
    code, neg = nearest_code(q.astype(np.float64), E2M1_POS)
    nib = code | (neg.astype(np.uint8) << 3)
    assert np.array_equal(c4[:2], nib[:, 0::2] | (nib[:, 1::2] << 4))


def test_nvfp4_at_the_edge_of_the_stated_domain(oracle):
    """Row scales 2^-100 and 2^+100 (the edge of the domain in which r~ and rho~ are normal binary32 numbers) and blocks
    whose E4M3 scale is subnormal or zero: the 2^k-shift invariance must hold bit for bit out to the edge, and the
    small blocks follow the definition (scale = nearest E4M3 value, codes = nearest E2M1 value of x * rho~ / scale)."""
    base = wl.bits(wl.make_inputs(wl.Workload("t", 6, 256, seed=33, outlier_frac=0.01))["x"])
    bv = bf16_vals(base).copy()
    bv[:, 16:32] *= np.float32(2.0 ** -5)       # a block whose scale a/6 lands in E4M3's subnormal range (below 2^-6)
    bv[:, 32:48] *= np.float32(2.0 ** -12)      # a block whose scale rounds to zero (a/6 < 2^-10): codes +-0
    base = bf16_bits(bv)
    c0, s0, r0 = oracle.mxnorm_nvfp4_ref(base)
    assert np.any((s0[:, 1] > 0) & (s0[:, 1] < 8)) and np.all(s0[:, 2] == 0) and np.all(c0[:, 16:24] & 0x77 == 0)
    for k in (-100, 100):
        xs = bf16_bits(bf16_vals(base) * np.float32(2.0 ** k))
        assert np.array_equal(bf16_vals(xs), bf16_vals(base) * np.float32(2.0 ** k))      # exact shift
        c1, s1, r1 = oracle.mxnorm_nvfp4_ref(xs)
        assert np.array_equal(c1, c0) and np.array_equal(s1, s0) and np.array_equal(r1, r0 * np.float32(2.0 ** k))
        c1, s1, r1 = oracle.mxnorm_ref(xs)
        cb, sb_, rb = oracle.mxnorm_ref(base)
        assert np.array_equal(c1, cb) and np.array_equal(s1, sb_) and np.array_equal(r1, rb * np.float32(2.0 ** k))
    # definition on the shifted rows (given r~)
    xs = bf16_bits(bf16_vals(base) * np.float32(2.0 ** -100))
    xv = bf16_vals(xs)
    c1, s1, r1 = oracle.mxnorm_nvfp4_ref(xs)
    rho = (np.float32(1.0) / r1).astype(np.float32)
    a = (np.abs(xv).reshape(6, -1, 16).max(-1) * rho[:, None]).astype(np.float32)
    sc, _ = nearest_code((a / np.float32(6.0)).astype(np.float32).astype(np.float64), E4M3_POS)
    assert np.array_equal(s1, sc)
    d = E4M3_POS[sc].astype(np.float32)
    with np.errstate(divide="ignore"):
        inv = np.where(d == 0, np.float32(0), (rho[:, None] / d).astype(np.float32))
    q = (xv * np.repeat(inv, 16, axis=1)).astype(np.float32)
    code, neg = nearest_code(q.astype(np.float64), E2M1_POS)
    nib = code | (neg.astype(np.uint8) << 3)
    assert np.array_equal(c1, nib[:, 0::2] | (nib[:, 1::2] << 4))


def test_nvfp4_scales_and_codes_by_definition_given_rho(oracle):
    x = wl.bits(wl.make_inputs(wl.Workload("t", 16, 512, seed=6, outlier_frac=0.004))["x"])
    xv = bf16_vals(x)
    for gs in (1.0, 4.0):
        codes, scales, r = oracle.mxnorm_nvfp4_ref(x, eps=1e-5, global_scale=gs)
        rho = (np.float32(1.0) / (r + np.float32(1e-5))).astype(np.float32)
        a = (np.abs(xv).reshape(16, -1, 16).max(-1) * rho[:, None]).astype(np.float32)
        t = ((a / np.float32(6.0)).astype(np.float32) * np.float32(gs)).astype(np.float32)
        sc, _ = nearest_code(t.astype(np.float64), E4M3_POS)
        assert np.array_equal(scales, sc)
        d = E4M3_POS[sc].astype(np.float32)
        with np.errstate(divide="ignore", invalid="ignore"):
            inv = np.where(d == 0, np.float32(0), ((rho * np.float32(gs)).astype(np.float32)[:, None] / d).astype(np.float32))
        q = (xv * np.repeat(inv, 16, axis=1)).astype(np.float32)
        code, neg = nearest_code(q.astype(np.float64), E2M1_POS)
        nib = code | (neg.astype(np.uint8) << 3)
        assert np.array_equal(codes, nib[:, 0::2] | (nib[:, 1::2] << 4))
        deq = E2M1_POS[code] * np.repeat(d, 16, axis=1) / gs
        ynorm = np.abs(xv * rho[:, None])
        # error <= half the widest E2M1 step (1.0) times the decoded scale d <= (a/6)(1+2^-4), plus the
        # saturation loss a*2^-4 when the E4M3 scale rounded down: <= 0.25*a in all
        assert np.all(np.abs(deq - ynorm) <= 0.25 * np.repeat(a, 16, axis=1) + 1e-6)


def test_plain_nvfp4_cast_by_definition(oracle):
    """The cast without a normaliser (weights): block scale = nearest E4M3 value to absmax/6*g, codes = nearest E2M1 value
    to x*g/scale, and it is what the normalising variants produce when their rho is 1."""
    x = wl.bits(wl.make_inputs(wl.Workload("t", 12, 256, seed=8, outlier_frac=0.004))["x"])
    xv = bf16_vals(x)
    for gs in (1.0, 0.5, 8.0):
        codes, scales = oracle.nvfp4_cast_ref(x, global_scale=gs)
        a = np.abs(xv).reshape(12, -1, 16).max(-1)
        t = ((a / np.float32(6.0)).astype(np.float32) * np.float32(gs)).astype(np.float32)
        sc, _ = nearest_code(t.astype(np.float64), E4M3_POS)
        assert np.array_equal(scales, sc)
        d = E4M3_POS[sc].astype(np.float32)
        with np.errstate(divide="ignore", invalid="ignore"):
            inv = np.where(d == 0, np.float32(0), (np.float32(gs) / d).astype(np.float32))
        q = (xv * np.repeat(inv, 16, axis=1)).astype(np.float32)
        code, neg = nearest_code(q.astype(np.float64), E2M1_POS)
        nib = code | (neg.astype(np.uint8) << 3)
        assert np.array_equal(codes, nib[:, 0::2] | (nib[:, 1::2] << 4))
    # a constant row of ones: absmax/6 = 0.16667 -> nearest E4M3 value 0.171875 = 0x23; 1/0.171875 = 5.818 -> 6 -> 0x7
    ones = np.full((1, 32), ONE, np.uint16)
    codes, scales = oracle.nvfp4_cast_ref(ones)
    assert np.all(scales == 0x23) and np.all(codes == 0x77)
    # the normalising variant with a coefficient that makes r~ = 1 exactly (constant row of ones: G = 1) gives the same bytes
    c2, s2, r2 = oracle.mxnorm_nvfp4_ref(ones, coef=1.0)
    assert r2[0] == 1.0 and np.array_equal(c2, codes) and np.array_equal(s2, scales)


def test_mxfp4_element_format_by_definition(oracle):
    """E2M1 values with E8M0 scales (the listing's cast with dtype = E2M1): the largest power of two of the
    format is 4, so S is the smallest power of two with absmax/S <= 4; codes are the nearest E2M1 values,
    two per byte (element 2i in the low nibble)."""
    E2 = oracle.ELEM_E2M1
    x = wl.bits(wl.make_inputs(wl.Workload("t", 20, 512, seed=12, outlier_frac=0.004))["x"])
    xv = bf16_vals(x)

    def check(codes, scales, y, B):
        m = np.abs(y).reshape(y.shape[0], -1, B).max(-1)
        sb = smallest_pow2_scale(m, emax=2)
        assert np.array_equal(scales, sb)
        S = np.repeat(np.ldexp(1.0, sb.astype(int) - 127), B, axis=1)
        code, neg = nearest_code(y.astype(np.float64) / S, E2M1_POS)
        nib = code | (neg.astype(np.uint8) << 3)
        assert np.array_equal(codes, nib[:, 0::2] | (nib[:, 1::2] << 4))

    for B in (16, 32, 64):
        codes, scales = oracle.mx_cast_ref(x, block=B, elem=E2)
        check(codes, scales, xv, B)
        codes, scales, r = oracle.mxnorm_ref(x, eps=1e-5, block=B, elem=E2)
        rho = (np.float32(1.0) / (r + np.float32(1e-5))).astype(np.float32)
        check(codes, scales, (xv * rho[:, None]).astype(np.float32), B)
        # the estimate does not depend on the element format
        assert np.array_equal(r, oracle.mxnorm_ref(x, eps=1e-5, block=B)[2])
        codes, scales, r = oracle.rmsnorm_mxfp8_ref(x, eps=1e-5, block=B, elem=E2)
        rho = (np.float32(1.0) / r).astype(np.float32)
        check(codes, scales, (xv * rho[:, None]).astype(np.float32), B)
    # constant row: x*rho~ = 2.389 in (2,4] -> S = 1 (biased 127), nearest E2M1 value 2 -> nibble 4 -> byte 0x44
    ones = np.full((2, 64), ONE, np.uint16)
    codes, scales, _ = oracle.mxnorm_ref(ones, elem=E2)
    assert np.all(scales == 127) and np.all(codes == 0x44)
    # 2^k shifts and all bf16 patterns as lone block maxima
    xs = bf16_bits(xv * np.float32(2.0 ** 5))
    c0, s0 = oracle.mx_cast_ref(x, elem=E2)
    c1, s1 = oracle.mx_cast_ref(xs, elem=E2)
    assert np.array_equal(c0, c1) and np.array_equal(s1.astype(int), s0.astype(int) + 5)
    pats = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    pats = pats[(pats & 0x7F80) != 0x7F80]
    xp = np.zeros((pats.size, 32), np.uint16)
    xp[:, 0] = pats
    xp[:, 1] = (pats >> 1) & 0x7FFF
    xp[(xp[:, 1] & 0x7F80) == 0x7F80, 1] = 0
    codes, scales = oracle.mx_cast_ref(xp, elem=E2)
    check(codes, scales, bf16_vals(xp), 32)


def test_transposed_cast_reduces_to_the_row_cast(oracle):
    """Blocks along the token axis of X are blocks along the last axis of X^T: without a normaliser the
    transposed cast equals mx_cast of the transposed matrix; with power-of-two row factors the scaled values
    stay exact bf16, so the same reduction pins the rho path; general rho is pinned by definition."""
    x = wl.bits(wl.make_inputs(wl.Workload("t", 96, 160, seed=14, outlier_frac=0.01))["x"])
    xv = bf16_vals(x)
    for B in (16, 32):
        ct, st = oracle.mx_cast_transposed_ref(x, block=B)
        c, s = oracle.mx_cast_ref(np.ascontiguousarray(x.T), block=B)
        assert np.array_equal(ct, c) and np.array_equal(st, s)
    # rho_t = 2^-k_t exactly (r = 2^k, eps = 0): scaled values are exact bf16
    k = np.random.default_rng(0).integers(-6, 7, size=96)
    r = np.ldexp(1.0, k).astype(np.float32)
    ys = bf16_bits(xv * np.ldexp(1.0, -k).astype(np.float32)[:, None])
    ct, st = oracle.mx_cast_transposed_ref(x, rms=r)
    c, s = oracle.mx_cast_ref(np.ascontiguousarray(ys.T))
    assert np.array_equal(ct, c) and np.array_equal(st, s)
    # general r (the MXNorm estimate) and eps: definitional check
    _, _, r_est = oracle.mxnorm_ref(x, eps=1e-5)
    ct, st = oracle.mx_cast_transposed_ref(x, rms=r_est, eps=1e-5)
    rho = (np.float32(1.0) / (r_est + np.float32(1e-5))).astype(np.float32)
    y = (xv * rho[:, None]).astype(np.float32).T                      # [D, T]
    m = np.abs(y).reshape(160, -1, 32).max(-1)
    sb = smallest_pow2_scale(m)
    assert np.array_equal(st, sb)
    code, neg = nearest_code(y.astype(np.float64) / np.repeat(np.ldexp(1.0, sb.astype(int) - 127), 32, axis=1), E4M3_POS)
    assert np.array_equal(ct, code | (neg.astype(np.uint8) << 7))
    # zero rms -> rho = 0 -> zero codes, zero scales
    ct, st = oracle.mx_cast_transposed_ref(x, rms=np.zeros(96, np.float32))
    assert np.all(st == 0) and np.all((ct & 0x7F) == 0)


def test_rmsnorm_nvfp4_by_definition(oracle):
    x = wl.bits(wl.make_inputs(wl.Workload("t", 16, 512, seed=21, outlier_frac=0.004))["x"])
    xv = bf16_vals(x)
    for gs, eps in ((1.0, 1e-5), (4.0, 0.0)):
        codes, scales, r = oracle.rmsnorm_nvfp4_ref(x, eps=eps, global_scale=gs)
        assert np.array_equal(r, oracle.rmsnorm_mxfp8_ref(x, eps=eps)[2])          # same r as Algorithm 1
        rho = (np.float32(1.0) / r).astype(np.float32)
        y = (xv * rho[:, None]).astype(np.float32)
        a = np.abs(y).reshape(16, -1, 16).max(-1)                                # absmax of the normalised values
        t = ((a / np.float32(6.0)).astype(np.float32) * np.float32(gs)).astype(np.float32)
        sc, _ = nearest_code(t.astype(np.float64), E4M3_POS)
        assert np.array_equal(scales, sc)
        d = E4M3_POS[sc].astype(np.float32)
        with np.errstate(divide="ignore", invalid="ignore"):
            inv = np.where(d == 0, np.float32(0), ((rho * np.float32(gs)).astype(np.float32)[:, None] / d).astype(np.float32))
        q = (xv * np.repeat(inv, 16, axis=1)).astype(np.float32)
        code, neg = nearest_code(q.astype(np.float64), E2M1_POS)
        nib = code | (neg.astype(np.uint8) << 3)
        assert np.array_equal(codes, nib[:, 0::2] | (nib[:, 1::2] << 4))
    # constant row: RMS = 1, x*rho = 1 -> scale E4M3(1/6 = 0.16667) = 0.171875 (0x23), q = 5.818 -> 6 -> 0x77
    codes, scales, r = oracle.rmsnorm_nvfp4_ref(np.full((2, 64), ONE, np.uint16))
    assert np.all(r == 1.0) and np.all(scales == 0x23) and np.all(codes == 0x77)


E5M2_POS = np.array([(m * 2.0 ** -16) if e == 0 else (4 + m) * 2.0 ** (e - 17)
                     for e in range(32) for m in range(4)][:0x7C], dtype=np.float64)   # codes 0..0x7B (57344)


def test_e5m2_element_format(oracle):
    """E5M2 (an option the paper names for gradients): encoder against brute force and torch's cast; the cast uses
    2^15, the largest power of two of the format, so block maxima land in (2^14, 2^15]."""
    assert E5M2_POS[-1] == 57344.0 and E5M2_POS[4] == 2.0 ** -14
    g = E5M2_POS
    mids = (g[:-1] + g[1:]) / 2
    probes = np.concatenate([g, mids, np.nextafter(mids.astype(np.float32), np.float32(0)),
                             np.nextafter(mids.astype(np.float32), np.float32(1e9)), [57344.0, 60000.0, 61440.0, 1e6, 2.0 ** -17, 1e-30]])
    probes = probes.astype(np.float32)
    want, _ = nearest_code(probes.astype(np.float64), g)
    got = np.array([oracle.e5m2_encode(float(v)) for v in probes], np.uint8)
    assert np.array_equal(got, want)
    assert oracle.e5m2_encode(-3.0) == (0x80 | oracle.e5m2_encode(3.0)) and oracle.e5m2_encode(float("inf")) == 0x7B
    rng = np.random.default_rng(0)
    v = np.concatenate([rng.standard_normal(20000) * 1000, rng.standard_normal(20000), rng.standard_normal(5000) * 1e-4]).astype(np.float32)
    v = v[np.abs(v) <= 57344.0]
    want = torch.from_numpy(v).to(torch.float8_e5m2).view(torch.uint8).numpy()
    got = np.array([oracle.e5m2_encode(float(a)) for a in v], np.uint8)
    assert np.array_equal(got, want)
    # the cast by definition
    x = wl.bits(wl.make_inputs(wl.Workload("t", 32, 256, seed=31, outlier_frac=0.01))["x"])
    xv = bf16_vals(x)
    codes, scales = oracle.mx_cast_ref(x, elem=oracle.ELEM_E5M2)
    m = np.abs(xv).reshape(32, -1, 32).max(-1)
    sb = smallest_pow2_scale(m, emax=15)
    assert np.array_equal(scales, sb)
    S = np.repeat(np.ldexp(1.0, sb.astype(int) - 127), 32, axis=1)
    code, neg = nearest_code(xv.astype(np.float64) / S, g)
    assert np.array_equal(codes, code | (neg.astype(np.uint8) << 7))
    top = (codes & 0x7F).reshape(32, -1, 32).max(-1)
    assert np.all((top >= 0x74) & (top <= 0x78))     # (2^14, 2^15], where values just above 2^14 round down to it
    ct, st = oracle.mx_cast_transposed_ref(x, elem=oracle.ELEM_E5M2)
    c2, s2 = oracle.mx_cast_ref(np.ascontiguousarray(x.T), elem=oracle.ELEM_E5M2)
    assert np.array_equal(ct, c2) and np.array_equal(st, s2)


def test_postround_estimator(oracle):
    """Post-round MXNorm: f(sigma) = E[max_i 2^floor(log2 |X_i|)] against Monte Carlo, the scaling identity
    f(2 sigma) = 2 f(sigma) the appendix states, f^-1 o f = id, and the estimator on Gaussian rows."""
    rng = np.random.default_rng(0)
    for B in (16, 32, 64):
        for sigma in (1.0, 0.37, 5.3):
            z = np.abs(rng.standard_normal((200000, B))) * sigma
            mc = np.exp2(np.floor(np.log2(z.max(-1)))).mean()
            f = oracle.postround_f(sigma, B)
            assert abs(f - mc) < 4e-3 * mc, (B, sigma, f, mc)
            assert abs(oracle.postround_f(2 * sigma, B) - 2 * f) < 1e-12 * f
            assert abs(oracle.postround_f_inverse(f, B) - sigma) < 1e-12 * sigma
        assert oracle.postround_f(1.0, B) < oracle.postround_f(1.01, B)          # increasing
    # estimator: r~ tracks the RMS of Gaussian rows (it is noisier than the pre-round estimator)
    x = wl.bits(wl.gaussian(512, 4096, seed=40, row_scale_sigma=1.0))
    xv = bf16_vals(x).astype(np.float64)
    rms = np.sqrt((xv ** 2).mean(-1))
    for B in (16, 32):
        codes, scales, r = oracle.mxnorm_postround_ref(x, block=B)
        ratio = r / rms
        assert abs(ratio.mean() - 1) < 0.01 and ratio.std() < 0.06, (B, ratio.mean(), ratio.std())
        # r~ = f^-1(mean of rounded absmaxes), re-derived with exact bisection instead of the table: within the
        # interpolation error of a 64-interval table
        m = np.abs(xv).reshape(512, -1, B).max(-1)
        xbar = np.exp2(np.floor(np.log2(m))).mean(-1)
        for t in (0, 17, 511):
            exact = oracle.postround_f_inverse(float(xbar[t]), B)
            assert abs(r[t] - exact) < 2e-3 * exact
        # scales and codes follow Algorithm 2 with this r~
        rho = (np.float32(1.0) / r).astype(np.float32)
        y = (bf16_vals(x) * rho[:, None]).astype(np.float32)
        sb = smallest_pow2_scale(np.abs(y).reshape(512, -1, B).max(-1))
        assert np.array_equal(scales, sb)
    # 2^k shift: xbar scales exactly, the table is scale free -> r~ scales exactly, codes and scales unchanged
    c0, s0, r0 = oracle.mxnorm_postround_ref(x[:32])
    xs = bf16_bits(bf16_vals(x[:32]) * np.float32(2.0 ** -7))
    c1, s1, r1 = oracle.mxnorm_postround_ref(xs)
    assert np.array_equal(c0, c1) and np.array_equal(s0, s1) and np.array_equal(r1, r0 * np.float32(2.0 ** -7))
    # eps enters as rho~ = 1/(r~ + eps): with eps = r~ the denominator doubles exactly, so every scale exponent
    # drops by one, the codes stay and the reported r~ does not include eps
    for t in (0, 5):
        c0, s0, r0 = oracle.mxnorm_postround_ref(x[t:t + 1])
        c1, s1, r1 = oracle.mxnorm_postround_ref(x[t:t + 1], eps=float(r0[0]))
        assert np.array_equal(r1, r0) and np.array_equal(c1, c0) and np.array_equal(s1.astype(int), s0.astype(int) - 1)
    z = np.zeros((1, 64), np.uint16)
    c, s_, r = oracle.mxnorm_postround_ref(z, eps=1e-5)
    assert np.all(c == 0) and np.all(s_ == 0) and r[0] == 0


def _scipy_postround_f(sigma, B):
    """E[max_i 2^floor(log2 |X_i|)] for B i.i.d. N(0, sigma^2) values, written from the definition with scipy:
    P(max rounds to 2^j) = P(max < 2^(j+1)) - P(max < 2^j), P(max < t) = erf(t / (sigma sqrt 2))^B, summed over a window of
    exponents far wider than any term that can matter in binary64."""
    from scipy import special
    j = np.arange(-300, 120, dtype=np.float64)
    cdf = special.erf(np.exp2(j) / (sigma * math.sqrt(2.0))) ** B
    cdf_next = special.erf(np.exp2(j + 1) / (sigma * math.sqrt(2.0))) ** B
    return float(np.sum(np.exp2(j) * (cdf_next - cdf)))


def test_postround_table_against_an_independent_restatement(oracle):
    """The post-round estimate r~ = f^-1(xbar): f rebuilt here with scipy's erf, inverted with scipy's brentq, tabulated at
    the 65 nodes 2^(i/64) of [1, 2], interpolated linearly in x with numpy, and scaled by f^-1(x) = 2^-k f^-1(2^k x) -
    the appendix' procedure with A = 64.  The oracle must agree to 1e-12 on random arguments, at the nodes, next to the
    wrap-around at 2 and at powers of two; and the table must stay within its interpolation error of exact inversion."""
    from scipy import optimize
    nodes = np.exp2(np.arange(65) / 64.0)
    nodes[64] = 2.0
    rng = np.random.default_rng(5)
    for B in (16, 32, 64):
        f = lambda s_: _scipy_postround_f(s_, B)
        # f itself (the oracle's series against the wide-window scipy sum) and f^-1 by bisection against brentq
        for sigma in (0.001, 0.37, 1.0, 1.9, 777.0):
            assert abs(oracle.postround_f(sigma, B) - f(sigma)) <= 1e-13 * f(sigma)
        values = np.array([optimize.brentq(lambda s_: f(s_) - x, x / 8, x * 4, xtol=1e-16, rtol=1e-15, maxiter=500) for x in nodes])
        for x, v in zip(nodes[::8], values[::8]):
            assert abs(oracle.postround_f_inverse(float(x), B) - v) <= 1e-12 * v
        assert np.all(np.diff(values) > 0)

        def restated(xbar):
            mant, ex = np.frexp(xbar)                        # xbar = mant * 2^ex, mant in [0.5, 1)
            z = 2.0 * mant
            return float(np.interp(z, nodes, values) * 2.0 ** (ex - 1))

        probes = list(np.exp(rng.uniform(np.log(1e-6), np.log(1e6), 300)))
        probes += [float(n) for n in nodes[:-1]] + [1.0, 2.0, 4.0, 0.5, 2.0 ** -40, 2.0 ** 37]
        probes += [float(np.nextafter(2.0, 0.0)), float(np.nextafter(1.0, 0.0)), float(np.nextafter(1.0, 2.0)),
                   float(np.nextafter(nodes[17], 0.0)), float(np.nextafter(nodes[17], 4.0)), 1.5 * 2.0 ** -20]
        got = oracle.postround_estimate(np.array(probes), B)
        want = np.array([restated(v) for v in probes])
        assert np.all(np.abs(got - want) <= 1e-12 * want), (B, np.max(np.abs(got - want) / want))
        exact = np.array([oracle.postround_f_inverse(v, B) for v in probes[:120]])
        worst = np.max(np.abs(got[:120] - exact) / exact)
        # 64 intervals, linear in x: the interpolation error grows with the block size (f gets more step-like);
        # measured 4e-5 / 1.5e-4 / 6.6e-4
        assert 1e-7 < worst < {16: 1e-4, 32: 3e-4, 64: 1.5e-3}[B], (B, worst)
        assert oracle.postround_estimate(0.0, B)[0] == 0.0
    # and the emitted binary32 r~ is that value rounded once
    x = wl.bits(wl.gaussian(64, 1024, seed=41, row_scale_sigma=1.0))
    xv = bf16_vals(x).astype(np.float64)
    for B in (16, 32, 64):
        _, _, r = oracle.mxnorm_postround_ref(x, block=B)
        m = np.abs(xv).reshape(64, -1, B).max(-1)
        xbar = np.exp2(np.floor(np.log2(m))).mean(-1)        # exact: powers of two, K a power of two
        assert np.array_equal(r, oracle.postround_estimate(xbar, B).astype(np.float32))


def test_residual_add_then_mxnorm(oracle):
    """h = bf16(x + res) must be torch's bf16 addition bit for bit, and the rest is Algorithm 2 on h."""
    a = wl.make_inputs(wl.Workload("t", 40, 512, seed=50, outlier_frac=0.004))["x"]
    b = wl.make_inputs(wl.Workload("t", 40, 512, seed=51))["x"] * 3
    b[3] = -a[3]                                              # exact cancellation -> a zero row
    b[4, ::2] = a[4, ::2] * 2.0 ** -12                          # tiny addends: rounding of the sum matters
    h, codes, scales, r = oracle.mxnorm_add_ref(wl.bits(a), wl.bits(b), eps=1e-5)
    assert np.array_equal(h, wl.bits(a + b))                  # torch adds bf16 tensors in fp32 and rounds once (RN-even)
    c2, s2, r2 = oracle.mxnorm_ref(h, eps=1e-5)
    assert np.array_equal(codes, c2) and np.array_equal(scales, s2) and np.array_equal(r, r2)
    assert r[3] == 0 and np.all(codes[3] & 0x7F == 0)


# ------------------------------------------------------------------ library restatements
def test_rms_estimate_against_numpy_restatement(oracle):
    x = _rand_rows(7, T=64, D=1024)
    xv = bf16_vals(x).astype(np.float64)
    for B in (16, 32, 64):
        for p in (1, 2):
            _, _, r = oracle.mxnorm_ref(x, p=p, block=B)
            m = np.abs(xv).reshape(64, -1, B).max(-1)
            G = (m ** p).mean(-1) ** (1.0 / p)
            want = np.float64(np.float32(oracle.coef(B, p))) * G
            assert np.all(np.abs(r - want) <= np.abs(want) * 2.0 ** -23)
    _, _, r = oracle.mxnorm_nvfp4_ref(x)
    m = np.abs(xv).reshape(64, -1, 16).max(-1)
    want = np.float64(np.float32(0.4688)) * np.sqrt((m ** 2).mean(-1))
    assert np.all(np.abs(r - want) <= np.abs(want) * 2.0 ** -23)


def test_rmsnorm_against_torch_rms_norm(oracle):
    x = _rand_rows(8, T=32, D=768)
    xt = torch.from_numpy(bf16_vals(x).astype(np.float64))
    for eps in (0.0, 1e-5):
        _, _, r = oracle.rmsnorm_mxfp8_ref(x, eps=eps)
        y = torch.nn.functional.rms_norm(xt, (768,), eps=eps)
        j = xt.abs().argmax(dim=-1)
        ratio = (xt[torch.arange(32), j] / y[torch.arange(32), j]).numpy()   # = sqrt(mean x^2 + eps)
        assert np.all(np.abs(r - ratio) <= ratio * 2.0 ** -23)


def test_e4m3_against_torch_cast(oracle):
    rng = np.random.default_rng(0)
    v = np.concatenate([rng.standard_normal(20000) * 100, rng.standard_normal(20000),
                        rng.standard_normal(5000) * 1e-2, [0.0, -0.0, 448.0, -448.0, 2.0 ** -9, 2.0 ** -10]])
    v = v.astype(np.float32)
    v = v[np.abs(v) <= 448.0]
    want = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([oracle.e4m3_encode(float(a)) for a in v], np.uint8)
    assert np.array_equal(got, want)


def test_e8m0_byte_is_the_biased_exponent(oracle):
    sb = np.array([0, 1, 100, 121, 127, 130, 254], np.uint8)
    vals = torch.from_numpy(sb).view(torch.float8_e8m0fnu).to(torch.float64).numpy()
    assert np.array_equal(vals, np.ldexp(1.0, sb.astype(int) - 127))
    for e in range(-126, 127):
        assert oracle.e8m0_scale(2.0 ** e) == max(0, e - 8 + 127)
        if e < 126:
            assert oracle.e8m0_scale(float(np.nextafter(np.float32(2.0 ** e), np.float32(np.inf)))) == max(0, e + 1 - 8 + 127)


# ------------------------------------------------------------------ P8: dequantisation error bound
def test_dequantisation_error_bound(oracle):
    x = wl.bits(wl.make_inputs(wl.Workload("t", 64, 2048, seed=9, outlier_frac=0.001))["x"])
    xv = bf16_vals(x).astype(np.float64)
    codes, scales, r = oracle.mxnorm_ref(x, eps=0.0)
    S = np.repeat(np.ldexp(1.0, scales.astype(int) - 127), 32, axis=1)
    mag = E4M3_POS[codes & 0x7F]
    deq = np.where(codes & 0x80, -mag, mag) * S
    y = xv / r[:, None].astype(np.float64)
    err = np.abs(deq - y)
    # half a unit in the 3-bit mantissa (2^-4 relative), or half the subnormal step S*2^-9, plus fp32 slack
    assert np.all(err <= np.maximum(np.abs(y) * 2.0 ** -4, S * 2.0 ** -10) * (1 + 1e-5))


def test_mxnorm_tracks_rmsnorm_on_gaussian_rows(oracle):
    # Section 3.6: scale/value distributions of MXNorm and RMSNorm+MXCast nearly coincide for Gaussian input
    x = wl.bits(wl.gaussian(256, 4096, seed=10, row_scale_sigma=1.0))
    c0, s0, r0 = oracle.rmsnorm_mxfp8_ref(x)
    c1, s1, r1 = oracle.mxnorm_ref(x)
    ratio = r1 / r0
    assert abs(ratio.mean() - 1) < 3e-3 and ratio.std() < 0.02     # ~1.35 % at K = 128
    assert np.mean(s0 == s1) > 0.9 and np.all(np.abs(s0.astype(int) - s1.astype(int)) <= 1)
    _, _, r16 = oracle.mxnorm_nvfp4_ref(x)
    assert abs((r16 / r0).mean() - 1) < 3e-3 and (r16 / r0).std() < 0.015
    x768 = wl.bits(wl.gaussian(1024, 768, seed=11, row_scale_sigma=1.0))
    ratio = oracle.mxnorm_ref(x768)[2] / oracle.rmsnorm_mxfp8_ref(x768)[2]
    assert abs(ratio.mean() - 1) < 4e-3 and 0.02 < ratio.std() < 0.04   # ~3 % at K = 24


# ------------------------------------------------------------------ P9: backward
def _rmsnorm_loss(xv, gam, w):
    r = np.sqrt((xv ** 2).mean(-1, keepdims=True))
    return float(((xv / r) * gam * w).sum())


def test_backward_against_finite_differences(oracle):
    rng = np.random.default_rng(0)
    T, D = 3, 64
    x = bf16_bits(rng.standard_normal((T, D)))
    g = bf16_bits(rng.standard_normal((T, D)))
    gain = bf16_bits(1 + 0.1 * rng.standard_normal(D))
    xv, gv, gam = (bf16_vals(a).astype(np.float64) for a in (x, g, gain))
    rms = np.sqrt((xv ** 2).mean(-1))
    # the oracle takes r as fp32: use rows whose RMS is an exact fp32 by feeding fp32-rounded r and
    # comparing against FD of the loss with that same fixed-precision r only through tolerance
    dx, dg = oracle.mxnorm_bwd_ref(x, g, gain, rms.astype(np.float32))
    h = 1e-6
    fd = np.zeros_like(xv)
    for t in range(T):
        for d in range(D):
            xp, xm = xv.copy(), xv.copy()
            xp[t, d] += h
            xm[t, d] -= h
            fd[t, d] = (_rmsnorm_loss(xp, gam, gv) - _rmsnorm_loss(xm, gam, gv)) / (2 * h)
    assert np.max(np.abs(dx - fd)) <= 2e-6 * np.max(np.abs(fd))   # fp32 rounding of r: 6e-8 relative, FD error ~1e-9
    fdg = np.zeros(D)
    for d in range(D):
        gp, gm = gam.copy(), gam.copy()
        gp[d] += h
        gm[d] -= h
        fdg[d] = (_rmsnorm_loss(xv, gp, gv) - _rmsnorm_loss(xv, gm, gv)) / (2 * h)
    assert np.max(np.abs(dg - fdg)) <= 2e-6 * np.max(np.abs(fdg))
    # no gain == gain of ones
    dx1, dg1 = oracle.mxnorm_bwd_ref(x, g, None, rms.astype(np.float32))
    dx2, dg2 = oracle.mxnorm_bwd_ref(x, g, np.full(D, ONE, np.uint16), rms.astype(np.float32))
    assert np.array_equal(dx1, dx2) and np.array_equal(dg1, dg2)


def test_backward_row_identities(oracle):
    rng = np.random.default_rng(1)
    T, D = 8, 256
    x = bf16_bits(rng.standard_normal((T, D)) * 3)
    g = bf16_bits(rng.standard_normal((T, D)) * 1e-2)
    gain = bf16_bits(1 + 0.1 * rng.standard_normal(D))
    xv, gv, gam = (bf16_vals(a).astype(np.float64) for a in (x, g, gain))
    true_rms = np.sqrt((xv ** 2).mean(-1))
    # with the true RMS the gradient is orthogonal to x (RMSNorm is scale invariant)
    dx, _ = oracle.mxnorm_bwd_ref(x, g, gain, true_rms.astype(np.float32))
    assert np.all(np.abs((dx * xv).sum(-1)) <= 1e-6 * np.abs(dx * xv).sum(-1))
    # straight-through with r~ != RMS: sum_d dX x = D * delta / r~ * (1 - RMS^2 / r~^2)
    _, _, r_est = oracle.mxnorm_ref(x)
    dx, dg = oracle.mxnorm_bwd_ref(x, g, gain, r_est)
    r = r_est.astype(np.float64)
    delta = (gv * gam * xv).mean(-1)
    want = D * delta / r * (1 - true_rms ** 2 / r ** 2)
    assert np.allclose((dx * xv).sum(-1), want, rtol=1e-9, atol=1e-12)
    assert np.allclose(dg, ((xv / r[:, None]) * gv).sum(0), rtol=1e-12, atol=1e-15)


def test_backward_zero_row_contributes_nothing(oracle):
    """A row of zeros (a padding token) has r~ = 0; the forward emits zeros for it whatever rho is, and the backward takes
    1/r = 0 there: dX of that row is 0, dgamma equals the sum over the other rows, everything finite."""
    rng = np.random.default_rng(2)
    T, D = 6, 128
    x = bf16_bits(rng.standard_normal((T, D)))
    x[2] = 0
    x[4, ::2] = 0x8000
    x[4, 1::2] = 0
    g = bf16_bits(rng.standard_normal((T, D)) * 1e-2)
    gain = bf16_bits(1 + 0.1 * rng.standard_normal(D))
    _, _, r = oracle.mxnorm_ref(x)
    assert r[2] == 0 and r[4] == 0 and np.all(r[[0, 1, 3, 5]] > 0)
    dx, dg = oracle.mxnorm_bwd_ref(x, g, gain, r)
    assert np.all(np.isfinite(dx)) and np.all(np.isfinite(dg))
    assert np.all(dx[2] == 0) and np.all(dx[4] == 0)
    keep = [0, 1, 3, 5]
    dx_k, dg_k = oracle.mxnorm_bwd_ref(x[keep], g[keep], gain, r[keep])
    assert np.array_equal(dx[keep], dx_k) and np.array_equal(dg, dg_k)


# ------------------------------------------------------------------ scale layout
def test_swizzle_is_a_tiled_bijection(oracle):
    for T, K in ((128, 4), (256, 24), (200, 6), (16, 128)):
        idx = oracle.swizzle_index_map(T, K)
        assert idx.shape == (T, K) and np.unique(idx).size == T * K and idx.max() < oracle.swizzle_bytes(T, K)
        for r, c in ((0, 0), (T - 1, K - 1), (min(T - 1, 33), min(K - 1, 5)), (min(T - 1, 127), 3)):
            assert idx[r, c] == oracle.swizzle_offset(r, c, K)
        # each 128-row x 4-column tile occupies one contiguous 512-byte slot; inside it 32 rows x 16 bytes,
        # the 16 bytes holding rows r, r+32, r+64, r+96 with 4 consecutive scales each
        assert np.array_equal(idx // 512, (np.arange(T)[:, None] // 128) * ((K + 3) // 4) + np.arange(K)[None, :] // 4)
        within = idx % 512
        assert np.array_equal(within // 16, np.broadcast_to((np.arange(T) % 32)[:, None], (T, K)))
        assert np.array_equal((within % 16) // 4, np.broadcast_to(((np.arange(T) % 128) // 32)[:, None], (T, K)))
        assert np.array_equal(within % 4, np.broadcast_to((np.arange(K) % 4)[None, :], (T, K)))
