/*
 * CPU oracle for the MXNorm hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the plain, slow, step-by-step statement of what the GPU library
 * must compute.  It shares no code, header, table or helper with the CUDA
 * path and must never be linked or called from it: only the test-suite, the
 * smoke check and the "cpu_baseline" / "--impl reference" legs of the
 * benchmark use it.  Host pointers only.
 *
 * Every function follows the paper's order of operations and notation:
 *   T rows (tokens), D hidden size, B block size, K = D/B blocks per row,
 *   m_tk block absmax, rho_t inverse RMS, S_tk block scale, V_tkb codes.
 * fl32(.) below means one IEEE binary32 round-to-nearest-even operation.
 * The file is compiled with -ffp-contract=off so that no multiply-add is
 * fused behind the text's back.
 *
 * Readings taken where the paper is silent or inconsistent are marked
 * [reading] where they are taken.
 *
 * Pin status (see tests/test_oracle_pins.py): every function and branch below is pinned by something other
 * than itself - the paper's printed constants and bounds, closed forms, invariants, brute-force definitional
 * searches, library special cases (torch casts, scipy's erf and root finder), finite differences.
 *   mx_cast_ref, rmsnorm_mxfp8_ref, mxnorm_ref (with and without gain), mxnorm_bwd_ref, mx_cast_transposed_ref,
 *   mxnorm_add_ref, mxnorm_postround_ref (series, inverse, table and interpolation against an independent
 *   scipy/numpy restatement) : pinned.
 *   mxnorm_nvfp4_ref, rmsnorm_nvfp4_ref, nvfp4_cast_ref : the paper gives only "B = 16, E2M1"; the scale rule is
 *     a stated reading, so these are PARITY UNPINNED BY THE PAPER and pinned by the definitional search,
 *     closed forms and invariants of that reading only.
 *   mxn_ref_swizzle_offset : the tiled scale layout is not in the paper; structural pin on the CPU, pinned
 *     against a block-scaled GEMM on the GPU.
 */
#include <float.h>
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- enums (values mirror the public ABI but are declared independently) -- */
enum { REF_ROUND_RCEIL_POW2 = 0, REF_ROUND_FLOOR_OCP = 1, REF_ROUND_RCEIL_MAX = 2 };
enum { REF_ELEM_E4M3 = 0, REF_ELEM_E2M1 = 1, REF_ELEM_E5M2 = 2 };

/* ------------------------------------------------------------------------- */
/* number formats (MXFP primer appendix; OCP MX element formats)              */
/* ------------------------------------------------------------------------- */

static float bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16; /* bf16 is the top half of a binary32: exact */
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* rho = 1/den in binary32, for the normalisation factors rho~ = 1/(r~ + eps) and rho = 1/r.
 * den == 0 gives 0 (a zero row stays zero) [reading].  A denominator so small that the
 * reciprocal would overflow binary32 (den < 2^-128: rows of subnormal magnitude) gives the
 * largest finite binary32 instead of infinity [reading: the reciprocal saturates, as the
 * element casts do], so that no 0 * inf = NaN can arise from finite input. */
static float recip_sat(float den)
{
    if (den == 0.0f) return 0.0f;
    float rho = 1.0f / den;
    return rho > FLT_MAX ? FLT_MAX : rho;
}

/* cast(q; E4M3): OCP "fn" flavour - bias 7, 3 mantissa bits, subnormals down to
 * 2^-9, largest finite 448 (0x7E), no infinities, NaN = 0x7F.  Round to nearest,
 * ties to the even mantissa; magnitudes that would round above 448 saturate to
 * 448 [reading: saturating cast]; the sign of zero is kept. */
static uint8_t e4m3_encode(float q)
{
    uint8_t sign = signbit(q) ? 0x80 : 0x00;
    if (isnan(q)) return sign | 0x7F;
    double a = fabs((double)q);
    if (a == 0.0) return sign;
    if (isinf(a)) return sign | 0x7E;
    int ex;
    (void)frexp(a, &ex);
    int e = ex - 1;                    /* floor(log2 a) */
    unsigned code;
    if (e < -6) {                      /* subnormal range: multiples of 2^-9 */
        double n = rint(ldexp(a, 9));  /* 0..8; 8 lands on the smallest normal */
        code = (unsigned)n;
    } else {
        double n = rint(ldexp(a, 3 - e)); /* a / 2^(e-3), in [8,16] */
        if (n == 16.0) { n = 8.0; e += 1; }
        if (e > 8) return sign | 0x7E;
        code = ((unsigned)(e + 7) << 3) | ((unsigned)n - 8u);
    }
    if (code > 0x7E) code = 0x7E;      /* 0x7F is NaN: saturate to 448 */
    return sign | (uint8_t)code;
}

static float e4m3_decode(uint8_t c)
{
    int ef = (c >> 3) & 0xF, mf = c & 7;
    double v = ef == 0 ? ldexp((double)mf, -9) : ldexp(8.0 + mf, ef - 7 - 3);
    return (float)((c & 0x80) ? -v : v);
}

/* cast(q; E5M2): OCP E5M2 - bias 15, 2 mantissa bits, subnormals down to 2^-16, largest finite 57344
 * (0x7B); 0x7C is infinity, 0x7D-0x7F NaN.  Round to nearest, ties to even; magnitudes that would round
 * above 57344 saturate to 57344 [reading: saturating cast]; the sign of zero is kept.  The paper names E5M2
 * as an option for gradient tensors (caption of the computational-graph figure). */
static uint8_t e5m2_encode(float q)
{
    uint8_t sign = signbit(q) ? 0x80 : 0x00;
    if (isnan(q)) return sign | 0x7F;
    double a = fabs((double)q);
    if (a == 0.0) return sign;
    if (isinf(a)) return sign | 0x7B;
    int ex;
    (void)frexp(a, &ex);
    int e = ex - 1;                       /* floor(log2 a) */
    unsigned code;
    if (e < -14) {                        /* subnormal range: multiples of 2^-16 */
        code = (unsigned)rint(ldexp(a, 16));   /* 0..4; 4 lands on the smallest normal */
    } else {
        double n = rint(ldexp(a, 2 - e)); /* a / 2^(e-2), in [4,8] */
        if (n == 8.0) { n = 4.0; e += 1; }
        if (e > 15) return sign | 0x7B;
        code = ((unsigned)(e + 15) << 2) | ((unsigned)n - 4u);
    }
    if (code > 0x7B) code = 0x7B;
    return sign | (uint8_t)code;
}

/* cast(q; E2M1): values {0, .5, 1, 1.5, 2, 3, 4, 6}; nibble code 0..7 plus sign
 * in bit 3; round to nearest, ties to the even code; saturate at 6. */
static uint8_t e2m1_encode(float q)
{
    uint8_t sign = signbit(q) ? 0x8 : 0x0;
    if (isnan(q)) return sign | 0x7; /* no NaN in the format [reading: saturate] */
    double a = fabs((double)q);
    unsigned code;
    if (a < 1.0) {
        code = (unsigned)rint(a * 2.0);           /* 0, .5, 1 -> 0,1,2 */
    } else if (isinf(a)) {
        code = 7;
    } else {
        int ex;
        (void)frexp(a, &ex);
        int e = ex - 1;                            /* floor(log2 a) >= 0 */
        if (e > 2) { code = 7; }
        else {
            double n = rint(ldexp(a, 1 - e));      /* a / 2^(e-1) in [2,4] */
            if (n == 4.0) { n = 2.0; e += 1; }
            code = e > 2 ? 7u : (((unsigned)(e + 1) << 1) | ((unsigned)n - 2u));
        }
    }
    if (code > 7) code = 7;
    return sign | (uint8_t)code;
}

/* largest power of two representable by the element format (Algorithm 1/2
 * caption: 256 for E4M3; 4 for E2M1), as a base-2 exponent */
static int elem_largest_pow2_exp(int elem) { return elem == REF_ELEM_E2M1 ? 2 : elem == REF_ELEM_E5M2 ? 15 : 8; }
static float elem_max(int elem) { return elem == REF_ELEM_E2M1 ? 6.0f : elem == REF_ELEM_E5M2 ? 57344.0f : 448.0f; }

/* ceil(log2 a) and floor(log2 a) of a positive finite binary32, exactly */
static int ceil_log2f(float a)
{
    int ex;
    float f = frexpf(a, &ex); /* a = f*2^ex, f in [0.5,1) */
    return f == 0.5f ? ex - 1 : ex;
}
static int floor_log2f(float a)
{
    int ex;
    (void)frexpf(a, &ex);
    return ex - 1;
}

/* cast(a / 2^emax; E8M0) (Eq. "S_tk = cast(m_tk/256; E8M0)"): the biased
 * exponent sb of the power-of-two scale S = 2^(sb-127).
 *   RCEIL_POW2 (paper's choice, RCEIL rounding applied to a/256): the smallest
 *               power of two S with a/S <= 2^emax, i.e. ceil(log2 a) - emax
 *   FLOOR_OCP : floor(log2 a) - emax (OCP MX specification)
 *   RCEIL_MAX : ceil(log2(a / max_elem)) with a/max_elem one fp32 division
 * A zero block gets sb = 0; sb is clamped to [0,254] (0xFF is NaN) [reading]. */
static uint8_t e8m0_scale(float a, int mode, int elem)
{
    if (!(a > 0.0f)) return 0;
    if (isinf(a)) return 254;
    int e;
    if (mode == REF_ROUND_FLOOR_OCP) {
        e = floor_log2f(a) - elem_largest_pow2_exp(elem);
    } else if (mode == REF_ROUND_RCEIL_MAX) {
        float t = a / elem_max(elem);
        if (!(t > 0.0f)) return 0;
        e = ceil_log2f(t);
    } else {
        e = ceil_log2f(a) - elem_largest_pow2_exp(elem);
    }
    int sb = e + 127;
    if (sb < 0) sb = 0;
    if (sb > 254) sb = 254;
    return (uint8_t)sb;
}

/* 2^(127-sb) as a binary32 (exact for every sb in [0,254]; 2^-127 is subnormal) */
static float inv_scale_f32(uint8_t sb) { return ldexpf(1.0f, 127 - (int)sb); }

static uint8_t elem_encode(float q, int elem)
{
    return elem == REF_ELEM_E2M1 ? e2m1_encode(q) : elem == REF_ELEM_E5M2 ? e5m2_encode(q) : e4m3_encode(q);
}

/* store one element code: E4M3 one byte per element; E2M1 two per byte,
 * element 2i in the low nibble and 2i+1 in the high nibble of byte i */
static void put_code(uint8_t *row_codes, int64_t d, uint8_t c, int elem)
{
    if (elem == REF_ELEM_E2M1) {
        uint8_t *p = row_codes + d / 2;
        if (d & 1) *p = (uint8_t)((*p & 0x0F) | (c << 4));
        else       *p = (uint8_t)((*p & 0xF0) | (c & 0x0F));
    } else {
        row_codes[d] = c;
    }
}
static int64_t code_row_bytes(int64_t D, int elem) { return elem == REF_ELEM_E2M1 ? D / 2 : D; }

/* Shared tail of Algorithms 1 and 2: given the fp32 normalised (and, when a
 * gain is given, gain-scaled) row y, take block absmaxes, E8M0 scales and codes:
 *   m_k = max_b |y_kb| ; S_k = cast(m_k / 2^emax; E8M0) ; V_kb = cast(y_kb / S_k). */
static void quantise_row(const float *y, int64_t D, int B, int mode, int elem,
                         uint8_t *row_codes, uint8_t *row_scales)
{
    int64_t K = D / B;
    for (int64_t k = 0; k < K; ++k) {
        float m = 0.0f;
        for (int b = 0; b < B; ++b) {
            float a = fabsf(y[k * B + b]);
            if (a > m) m = a;
        }
        uint8_t sb = e8m0_scale(m, mode, elem);
        row_scales[k] = sb;
        float inv = inv_scale_f32(sb);
        for (int b = 0; b < B; ++b) {
            float q = y[k * B + b] * inv; /* y / S : scaling by a power of two */
            put_code(row_codes, k * B + b, elem_encode(q, elem), elem);
        }
    }
}

static int shape_ok(int64_t T, int64_t D, int B)
{
    return T >= 0 && D > 0 && (B == 16 || B == 32 || B == 64) && D % B == 0;
}

/* ------------------------------------------------------------------------- */
/* O1  MXCast (Section "Conversion to MXFP8 (MXCast)", Eqs. for S_tk, V_tkb)   */
/* ------------------------------------------------------------------------- */
int mx_cast_ref(const uint16_t *x_bf16, int64_t T, int64_t D, int B, int mode, int elem,
                uint8_t *codes, uint8_t *scales)
{
    if (!shape_ok(T, D, B)) return 1;
    int64_t K = D / B, cb = code_row_bytes(D, elem);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        float y[D];
        for (int64_t d = 0; d < D; ++d) y[d] = bf16_to_f32(x_bf16[t * D + d]);
        quantise_row(y, D, B, mode, elem, codes + t * cb, scales + t * K);
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* O2  Algorithm 1: RMSNorm + MXCast (Section "RMSNorm", Eqs. rho_t, Y_td)     */
/*     ms = (1/D) sum x^2 in fp64; r = fl32(sqrt(ms + eps)); rho = fl32(1/r);  */
/*     y = fl32(x*rho), then y = fl32(y*gamma) when a gain is given (gain      */
/*     before the cast, Eq. Y_td); no bf16 rounding between norm and cast      */
/*     [reading: "fused into a single kernel"].  Emits r.                      */
/* ------------------------------------------------------------------------- */
int rmsnorm_mxfp8_ref(const uint16_t *x_bf16, const uint16_t *gain_bf16, int64_t T, int64_t D,
                      int B, float eps, int mode, int elem,
                      uint8_t *codes, uint8_t *scales, float *rms_out)
{
    if (!shape_ok(T, D, B)) return 1;
    int64_t K = D / B, cb = code_row_bytes(D, elem);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        const uint16_t *xr = x_bf16 + t * D;
        double ss = 0.0;
        for (int64_t d = 0; d < D; ++d) {
            double v = (double)bf16_to_f32(xr[d]);
            ss += v * v;
        }
        double ms = ss / (double)D;
        float r = (float)sqrt(ms + (double)eps);
        float rho = recip_sat(r);
        float y[D];
        for (int64_t d = 0; d < D; ++d) {
            float v = bf16_to_f32(xr[d]) * rho;
            if (gain_bf16) v = v * bf16_to_f32(gain_bf16[d]);
            y[d] = v;
        }
        quantise_row(y, D, B, mode, elem, codes + t * cb, scales + t * K);
        if (rms_out) rms_out[t] = r;
    }
    return 0;
}

/* correction constant  RMS / G_p  for i.i.d. Gaussian blocks, as printed in the
 * paper's implementation appendix (4 digits).  Returns 0 for unknown (B,p). */
float mxn_ref_coef(int B, int p)
{
    if (B == 16 && p == 1) return 0.4814f;
    if (B == 16 && p == 2) return 0.4688f;
    if (B == 32 && p == 1) return 0.4261f;
    if (B == 32 && p == 2) return 0.4185f;
    if (B == 64 && p == 1) return 0.3852f;
    if (B == 64 && p == 2) return 0.3803f;
    return 0.0f;
}

/* steps 1-3 of Algorithm 2 for one row: block absmaxes m_k (exact), the
 * generalised p-mean G = (1/K sum m_k^p)^(1/p) in fp64 (Eq. G_K^(p)), the RMS
 * estimate r~ = fl32(coef * G) [reading: coef = RMS/G < 1 multiplies G], and
 * rho~ = fl32(1 / fl32(r~ + eps)), 0 when the denominator is 0 and saturating at the largest
 * finite binary32 (recip_sat) [reading]. */
static void mxnorm_row_stat(const uint16_t *xr, int64_t D, int B, int p, float coef, float eps,
                            float *m /* [K] */, float *r_est, float *rho)
{
    int64_t K = D / B;
    double s = 0.0;
    for (int64_t k = 0; k < K; ++k) {
        float mk = 0.0f;
        for (int b = 0; b < B; ++b) {
            float a = fabsf(bf16_to_f32(xr[k * B + b]));
            if (a > mk) mk = a;
        }
        m[k] = mk;
        s += p == 1 ? (double)mk : (double)mk * (double)mk;
    }
    double G = p == 1 ? s / (double)K : sqrt(s / (double)K);
    float rt = (float)((double)coef * G);
    float den = rt + eps;
    *r_est = rt;
    *rho = recip_sat(den);
}

/* ------------------------------------------------------------------------- */
/* O3  Algorithm 2: MXNorm (Section "MXNorm", Eqs. m~, rho~, S~, V~)           */
/*     a_k = fl32(m_k * rho~) ; S~_k = cast(a_k / 2^emax; E8M0) ;              */
/*     V~_kb = cast(fl32(x_kb * rho~) / S~_k).  Because fl32 is monotone,      */
/*     a_k equals the block absmax of fl32(x * rho~), so the shared tail is    */
/*     used.  With a gain (an extension, not in the paper: the paper folds     */
/*     the gain into the next weight) scales and codes are taken from          */
/*     fl32(fl32(x*rho~)*gamma) while rho~ still comes from |x|.  Emits r~.    */
/* ------------------------------------------------------------------------- */
int mxnorm_ref(const uint16_t *x_bf16, const uint16_t *gain_bf16, int64_t T, int64_t D,
               int B, int p, float coef, float eps, int mode, int elem,
               uint8_t *codes, uint8_t *scales, float *rms_est_out)
{
    if (!shape_ok(T, D, B) || (p != 1 && p != 2)) return 1;
    if (coef == 0.0f) coef = mxn_ref_coef(B, p);
    int64_t K = D / B, cb = code_row_bytes(D, elem);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        const uint16_t *xr = x_bf16 + t * D;
        float m[K], y[D];
        float r_est, rho;
        mxnorm_row_stat(xr, D, B, p, coef, eps, m, &r_est, &rho);
        for (int64_t d = 0; d < D; ++d) {
            float v = bf16_to_f32(xr[d]) * rho;
            if (gain_bf16) v = v * bf16_to_f32(gain_bf16[d]);
            y[d] = v;
        }
        quantise_row(y, D, B, mode, elem, codes + t * cb, scales + t * K);
        if (rms_est_out) rms_est_out[t] = r_est;
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* O4  NVFP4 variant of MXNorm [reading - the paper says only "B=16, E2M1"]:   */
/*     steps 1-3 with B = 16; a_k = fl32(m_k*rho~);                            */
/*     t_k = fl32(fl32(a_k / 6) * global_scale); block scale = cast(t_k; E4M3) */
/*     (6 = largest E2M1 value); d_k = the decoded scale;                      */
/*     inv_k = fl32(fl32(rho~ * global_scale) / d_k) (0 when d_k = 0), saturating */
/*     at the largest finite binary32 [reading, as for rho~ itself: a quotient  */
/*     that overflowed to infinity would turn zero elements into NaN];         */
/*     V_kb = cast(fl32(x_kb * inv_k); E2M1), two codes per byte.              */
/* ------------------------------------------------------------------------- */
/* shared NVFP4 tail: given the row's block absmaxes m_k of |x| and rho, emit E4M3 block scales and E2M1 codes */
static void nvfp4_quantise_row(const uint16_t *xr, const float *m, int64_t D, float rho, float global_scale,
                               uint8_t *row_codes, uint8_t *row_scales)
{
    const int B = 16;
    int64_t K = D / B;
    float rho_g = rho * global_scale;
    for (int64_t k = 0; k < K; ++k) {
        float a = m[k] * rho;
        float tk = (a / 6.0f) * global_scale;
        uint8_t sc = e4m3_encode(tk);
        row_scales[k] = sc;
        float dk = e4m3_decode(sc);
        float inv = dk == 0.0f ? 0.0f : rho_g / dk;
        if (inv > FLT_MAX) inv = FLT_MAX;
        for (int b = 0; b < B; ++b) {
            float q = bf16_to_f32(xr[k * B + b]) * inv;
            put_code(row_codes, k * B + b, e2m1_encode(q), REF_ELEM_E2M1);
        }
    }
}

int mxnorm_nvfp4_ref(const uint16_t *x_bf16, int64_t T, int64_t D, int p, float coef, float eps,
                     float global_scale, uint8_t *codes_packed, uint8_t *scales_e4m3,
                     float *rms_est_out)
{
    const int B = 16;
    if (!shape_ok(T, D, B) || (p != 1 && p != 2)) return 1;
    if (coef == 0.0f) coef = mxn_ref_coef(B, p);
    int64_t K = D / B;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        const uint16_t *xr = x_bf16 + t * D;
        float m[K];
        float r_est, rho;
        mxnorm_row_stat(xr, D, B, p, coef, eps, m, &r_est, &rho);
        nvfp4_quantise_row(xr, m, D, rho, global_scale, codes_packed + t * (D / 2), scales_e4m3 + t * K);
        if (rms_est_out) rms_est_out[t] = r_est;
    }
    return 0;
}

/* The plain NVFP4 cast (no normalisation: rho = 1), e.g. of a weight matrix: the tail above applied to x itself
 * [reading, as above; a per-tensor global_scale is the caller's]. */
int nvfp4_cast_ref(const uint16_t *x_bf16, int64_t T, int64_t D, float global_scale,
                   uint8_t *codes_packed, uint8_t *scales_e4m3)
{
    const int B = 16;
    if (!shape_ok(T, D, B)) return 1;
    int64_t K = D / B;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        const uint16_t *xr = x_bf16 + t * D;
        float m[K];
        for (int64_t k = 0; k < K; ++k) {
            float mk = 0.0f;
            for (int b = 0; b < B; ++b) {
                float a = fabsf(bf16_to_f32(xr[k * B + b]));
                if (a > mk) mk = a;
            }
            m[k] = mk;
        }
        nvfp4_quantise_row(xr, m, D, 1.0f, global_scale, codes_packed + t * (D / 2), scales_e4m3 + t * K);
    }
    return 0;
}

/* The conventional counterpart in the same format: Algorithm 1's rho (true RMS) followed by the NVFP4 cast of
 * x * rho [reading, as above].  Block absmaxes of fl32(x*rho) equal fl32(m_k * rho) because rounding is monotone. */
int rmsnorm_nvfp4_ref(const uint16_t *x_bf16, int64_t T, int64_t D, float eps, float global_scale,
                      uint8_t *codes_packed, uint8_t *scales_e4m3, float *rms_out)
{
    const int B = 16;
    if (!shape_ok(T, D, B)) return 1;
    int64_t K = D / B;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        const uint16_t *xr = x_bf16 + t * D;
        float m[K];
        double ss = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            float mk = 0.0f;
            for (int b = 0; b < B; ++b) {
                float v = bf16_to_f32(xr[k * B + b]);
                ss += (double)v * (double)v;
                if (fabsf(v) > mk) mk = fabsf(v);
            }
            m[k] = mk;
        }
        float r = (float)sqrt(ss / (double)D + (double)eps);
        float rho = recip_sat(r);
        nvfp4_quantise_row(xr, m, D, rho, global_scale, codes_packed + t * (D / 2), scales_e4m3 + t * K);
        if (rms_out) rms_out[t] = r;
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* O5  Backward (appendix "RMSNorm gradients"), straight-through: the RMSNorm  */
/*     gradient evaluated with whatever r the forward saved (r~ for MXNorm).   */
/*     g is the gradient w.r.t. Z = (X/r) gamma.  All in fp64.                 */
/*       dgamma_j = sum_t (x_tj / r_t) g_tj                                    */
/*       h = g * gamma ; delta_t = (1/D) sum_d h_td x_td                       */
/*       dX_td = h_td / r_t - x_td * delta_t / r_t^3                           */
/*     A row whose saved r is 0 is a row of zeros (r~ = 0 only when every      */
/*     block absmax is 0), for which the forward emitted zeros whatever rho    */
/*     was: 1/r is taken as 0 there, so the row contributes nothing to dgamma  */
/*     and gets dX = 0 [reading: the forward's "zero denominator -> rho = 0"]. */
/* ------------------------------------------------------------------------- */
int mxnorm_bwd_ref(const uint16_t *x_bf16, const uint16_t *g_bf16, const uint16_t *gain_bf16,
                   const float *rms, int64_t T, int64_t D, double *dx, double *dgain)
{
    if (T < 0 || D <= 0) return 1;
    /* dX: rows are independent */
    if (dx) {
#pragma omp parallel for schedule(static)
        for (int64_t t = 0; t < T; ++t) {
            const uint16_t *xr = x_bf16 + t * D, *gr = g_bf16 + t * D;
            double r = (double)rms[t];
            if (r == 0.0) {   /* zero row: see the note above */
                for (int64_t d = 0; d < D; ++d) dx[t * D + d] = 0.0;
                continue;
            }
            double dot = 0.0;
            for (int64_t d = 0; d < D; ++d) {
                double gam = gain_bf16 ? (double)bf16_to_f32(gain_bf16[d]) : 1.0;
                double h = (double)bf16_to_f32(gr[d]) * gam;
                dot += h * (double)bf16_to_f32(xr[d]);
            }
            double delta = dot / (double)D;
            for (int64_t d = 0; d < D; ++d) {
                double x = (double)bf16_to_f32(xr[d]);
                double gam = gain_bf16 ? (double)bf16_to_f32(gain_bf16[d]) : 1.0;
                double h = (double)bf16_to_f32(gr[d]) * gam;
                dx[t * D + d] = h / r - x * delta / (r * r * r);
            }
        }
    }
    /* dgamma: the column sum over the rows, in row order, kept a plain serial loop */
    if (dgain) {
        for (int64_t d = 0; d < D; ++d) dgain[d] = 0.0;
        for (int64_t t = 0; t < T; ++t) {
            double r = (double)rms[t];
            if (r == 0.0) continue;
            for (int64_t d = 0; d < D; ++d)
                dgain[d] += ((double)bf16_to_f32(x_bf16[t * D + d]) / r) * (double)bf16_to_f32(g_bf16[t * D + d]);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* O8  Residual add fused in front of MXNorm (pre-norm transformer blocks add  */
/*     the residual branch right before the norm; the layer benchmark of the   */
/*     paper notes that this add is fused with the norm).                      */
/*     h = bf16(fl32(x) + fl32(res)) (round-to-nearest-even to bf16), written  */
/*     out as the new residual stream; then Algorithm 2 on h.                  */
/* ------------------------------------------------------------------------- */
static uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040); /* NaN stays NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

int mxnorm_add_ref(const uint16_t *x_bf16, const uint16_t *res_bf16, int64_t T, int64_t D, int B, int p, float coef,
                   float eps, int mode, uint16_t *h_bf16, uint8_t *codes, uint8_t *scales, float *rms_est_out)
{
    if (!shape_ok(T, D, B) || (p != 1 && p != 2)) return 1;
    for (int64_t i = 0; i < T * D; ++i) h_bf16[i] = f32_to_bf16_rne(bf16_to_f32(x_bf16[i]) + bf16_to_f32(res_bf16[i]));
    return mxnorm_ref(h_bf16, NULL, T, D, B, p, coef, eps, mode, REF_ELEM_E4M3, codes, scales, rms_est_out);
}

/* ------------------------------------------------------------------------- */
/* O7  Post-round MXNorm (appendix "Post-round MXNorm"): the RMS is estimated    */
/*     from the block absmaxes AFTER rounding them to powers of two,            */
/*       s_k = r(m_k) = 2^floor(log2 m_k)   (0 for a zero block),                */
/*       xbar = (1/K) sum_k s_k,   r~ = f^-1(xbar),                              */
/*     where f(sigma) = E[max_i r(X_i)] for B i.i.d. N(0, sigma^2) values:       */
/*       f(sigma) = sum_j 2^j [ P(2^(j+1)) - P(2^j) ],  P(t) = erf(t/(sigma sqrt2))^B */
/*     [reading: the printed series has the two terms in the other order, which  */
/*     would make the expectation negative].  f^-1 is evaluated as the appendix  */
/*     describes: a table of f^-1(2^(i/A)), i = 0..A, linear interpolation in x  */
/*     on [1,2], and f^-1(x) = 2^-k f^-1(2^k x) elsewhere [reading: A = 64; the  */
/*     paper leaves A open].  Scales and codes then follow Algorithm 2 with this */
/*     r~.  PARITY UNPINNED by printed values: pinned by f(2s) = 2f(s), a Monte  */
/*     Carlo estimate of f, f^-1(f(s)) = s and the estimator's mean on Gaussian  */
/*     rows.                                                                     */
/* ------------------------------------------------------------------------- */
#define POSTROUND_A 64

static double postround_f(double sigma, int B)
{
    /* terms are negligible below 2^-60 sigma (P ~ 0) and above 2^5 sigma (P(2^j) = 1 to the last bit) */
    int j0 = (int)floor(log2(sigma));
    double sum = 0.0;
    for (int j = j0 - 64; j <= j0 + 6; ++j) {
        double lo = erf(ldexp(1.0, j) / (sigma * 1.4142135623730951));
        double hi = erf(ldexp(1.0, j + 1) / (sigma * 1.4142135623730951));
        sum += ldexp(1.0, j) * (pow(hi, B) - pow(lo, B));
    }
    return sum;
}

static double postround_f_inverse(double x, int B)
{
    /* f is increasing and f(sigma) lies between 0.5 sigma and 4 sigma for B in 16..64: bisect */
    double lo = x / 8.0, hi = x * 4.0;
    for (int it = 0; it < 200; ++it) {
        double mid = 0.5 * (lo + hi);
        if (postround_f(mid, B) < x) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

static void postround_table(int B, double *nodes, double *values)
{
    for (int i = 0; i <= POSTROUND_A; ++i) {
        nodes[i] = exp2((double)i / POSTROUND_A);
        values[i] = postround_f_inverse(nodes[i], B);
    }
    nodes[POSTROUND_A] = 2.0;
}

static double postround_estimate(double xbar, const double *nodes, const double *values)
{
    if (!(xbar > 0.0)) return 0.0;
    int ex;
    double z = 2.0 * frexp(xbar, &ex); /* xbar = z * 2^(ex-1), z in [1,2) */
    int i = 0;
    while (i + 1 < POSTROUND_A && nodes[i + 1] <= z) ++i; /* nodes[i] <= z < nodes[i+1] */
    double v = values[i] + (z - nodes[i]) * ((values[i + 1] - values[i]) / (nodes[i + 1] - nodes[i]));
    return ldexp(v, ex - 1);
}

double mxn_ref_postround_f(double sigma, int B) { return postround_f(sigma, B); }
double mxn_ref_postround_f_inverse(double x, int B) { return postround_f_inverse(x, B); }
/* the table-based estimates r~ = f^-1(xbar[i]) exactly as mxnorm_postround_ref evaluates them, before the rounding
 * to binary32 (the table is built once per call) */
void mxn_ref_postround_estimate(const double *xbar, int64_t n, int B, double *out)
{
    double nodes[POSTROUND_A + 1], values[POSTROUND_A + 1];
    postround_table(B, nodes, values);
    for (int64_t i = 0; i < n; ++i) out[i] = postround_estimate(xbar[i], nodes, values);
}

int mxnorm_postround_ref(const uint16_t *x_bf16, int64_t T, int64_t D, int B, float eps, int mode,
                         uint8_t *codes, uint8_t *scales, float *rms_est_out)
{
    if (!shape_ok(T, D, B)) return 1;
    int64_t K = D / B;
    double nodes[POSTROUND_A + 1], values[POSTROUND_A + 1];
    postround_table(B, nodes, values);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        const uint16_t *xr = x_bf16 + t * D;
        float y[D];
        double s = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            float mk = 0.0f;
            for (int b = 0; b < B; ++b) {
                float a = fabsf(bf16_to_f32(xr[k * B + b]));
                if (a > mk) mk = a;
            }
            if (mk > 0.0f) s += ldexp(1.0, floor_log2f(mk));
        }
        float rt = (float)postround_estimate(s / (double)K, nodes, values);
        float den = rt + eps;
        float rho = recip_sat(den);
        for (int64_t d = 0; d < D; ++d) y[d] = bf16_to_f32(xr[d]) * rho;
        quantise_row(y, D, B, mode, REF_ELEM_E4M3, codes + t * D, scales + t * K);
        if (rms_est_out) rms_est_out[t] = rt;
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* O6  Column-wise (transposed) MXCast for the weight-gradient GEMM            */
/*     (Section "MXNormLinear": grad W = MXCast(grad H^T) MXCast(rho~ X) gamma,*/
/*     where the activation must be block-quantised along the TOKEN axis).     */
/*     y_td = fl32(x_td * rho_t), rho_t = fl32(1 / fl32(r_t + eps)) (0 when    */
/*     the denominator is 0) or 1 when no r is given; blocks are B consecutive */
/*     tokens of one column; S, V as in MXCast; outputs are laid out           */
/*     transposed: codes [D, T], scales [D, T/B].                              */
/* ------------------------------------------------------------------------- */
int mx_cast_transposed_ref(const uint16_t *x_bf16, const float *rms_or_null, int64_t T, int64_t D, int B,
                           float eps, int mode, int elem, uint8_t *codes_t, uint8_t *scales_t)
{
    if (elem == REF_ELEM_E2M1) return 1;   /* one byte per element only */
    if (T < 0 || D <= 0 || !(B == 16 || B == 32 || B == 64) || T % B != 0) return 1;
    int64_t KT = T / B;
#pragma omp parallel for schedule(static)
    for (int64_t d = 0; d < D; ++d) {
        for (int64_t k = 0; k < KT; ++k) {
            float y[64];
            float m = 0.0f;
            for (int b = 0; b < B; ++b) {
                int64_t t = k * B + b;
                float rho = 1.0f;
                if (rms_or_null) {
                    float den = rms_or_null[t] + eps;
                    rho = recip_sat(den);
                }
                y[b] = bf16_to_f32(x_bf16[t * D + d]) * rho;
                float a = fabsf(y[b]);
                if (a > m) m = a;
            }
            uint8_t sb = e8m0_scale(m, mode, elem);
            scales_t[d * KT + k] = sb;
            float inv = inv_scale_f32(sb);
            for (int b = 0; b < B; ++b) codes_t[d * T + k * B + b] = elem_encode(y[b] * inv, elem);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* helpers exported for the tests                                             */
/* ------------------------------------------------------------------------- */

/* Byte offset of scale (row r, block c) in the 128x4-tiled layout that block-
 * scaled tensor-core GEMMs read [reading - not in the paper]: rows padded to a
 * multiple of 128, scale columns to a multiple of 4; each 128-row x 4-column
 * tile is 512 contiguous bytes, tiles ordered row-tile major. */
int64_t mxn_ref_swizzle_offset(int64_t r, int64_t c, int64_t K)
{
    int64_t tiles_per_row = (K + 3) / 4;
    int64_t tile = (r / 128) * tiles_per_row + c / 4;
    int64_t rr = r % 128;
    return tile * 512 + (rr % 32) * 16 + (rr / 32) * 4 + (c % 4);
}
int64_t mxn_ref_swizzle_bytes(int64_t T, int64_t K)
{
    return ((T + 127) / 128) * ((K + 3) / 4) * 512;
}

uint8_t mxn_ref_e4m3_encode(float q) { return e4m3_encode(q); }
float   mxn_ref_e4m3_decode(uint8_t c) { return e4m3_decode(c); }
uint8_t mxn_ref_e2m1_encode(float q) { return e2m1_encode(q); }
uint8_t mxn_ref_e5m2_encode(float q) { return e5m2_encode(q); }
uint8_t mxn_ref_e8m0_scale(float a, int mode, int elem) { return e8m0_scale(a, mode, elem); }

int mxn_ref_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
