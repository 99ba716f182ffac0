// Per-row device code shared by the forward kernels: the row statistic and its finishing step, block
// absmaxes, scale addressing, and the quantise-and-store phases for E4M3/E5M2, MXFP4 and NVFP4 outputs.
// Included by every translation unit that normalises rows (the constant-memory tables below are private
// to each of them; only the one that launches the post-round variant fills its copy).
#ifndef MXN_ROW_CUH_
#define MXN_ROW_CUH_

#include "mxn_device.cuh"
#include "mxn_internal.h"

namespace mxn {

#ifndef MXN_FWD_WARPS
#define MXN_FWD_WARPS 4          // warps per CTA (more when one row needs more); rows per CTA = warps / WPR
#endif
#ifndef MXN_FWD_MAX_ELEMS
#define MXN_FWD_MAX_ELEMS 64     // elements a lane holds per row (registers: half as many 32-bit words)
#endif
#ifndef MXN_FWD_MIN_CTAS
#define MXN_FWD_MIN_CTAS 1       // occupancy hint for the register allocator
#endif

// warps of a CTA whose rows each span WPR warps
__host__ __device__ constexpr int rows_per_cta(int wpr) { return MXN_FWD_WARPS / wpr > 1 ? MXN_FWD_WARPS / wpr : 1; }
__host__ __device__ constexpr int cta_warps(int wpr) { return wpr * rows_per_cta(wpr); }
// occupancy hint: the kernels are held to 64 registers per thread, i.e. 32 warps per SM whatever the CTA
// size (one register more is allocated as 72: a four-warp CTA then fits 7 times instead of 8, an eight-warp CTA 3 times
// instead of 4, a sixteen-warp CTA once instead of twice)
__host__ __device__ constexpr int fwd_min_ctas(int wpr) { return 32 / cta_warps(wpr); }

// ---- post-round estimator tables (appendix "Post-round MXNorm") ------------------------------------
// f^-1 sampled at the 65 nodes 2^(i/64) of [1,2] for each block size, with the slope of every interval;
// filled by postround_prepare() on the host, read by finish_stat<STAT_POSTROUND>.
constexpr int kPrIntervals = 64;
static __device__ __constant__ double c_pr_nodes[kPrIntervals + 1];
static __device__ __constant__ double c_pr_values[3][kPrIntervals + 1];
static __device__ __constant__ double c_pr_slopes[3][kPrIntervals];

__device__ __forceinline__ double postround_estimate(double xbar, int table)
{
    if (!(xbar > 0.0)) return 0.0;
    const unsigned long long bits = (unsigned long long)__double_as_longlong(xbar);
    const int e = (int)((bits >> 52) & 0x7FFull) - 1023;
    const double z = __longlong_as_double((long long)((bits & 0x000FFFFFFFFFFFFFull) | 0x3FF0000000000000ull));   // in [1,2)
    int i = 0;
#pragma unroll
    for (int step = kPrIntervals / 2; step >= 1; step >>= 1)
        if (c_pr_nodes[i + step] <= z) i += step;        // nodes[i] <= z < nodes[i+1]
    const double v = __dadd_rn(c_pr_values[table][i], __dmul_rn(__dadd_rn(z, -c_pr_nodes[i]), c_pr_slopes[table][i]));
    const double pow2 = __longlong_as_double((long long)(unsigned long long)(e + 1023) << 52);
    return __dmul_rn(v, pow2);
}

// row statistic -> (r, rho) ; one value per row group ------------------------------------------
template <int STAT>
__device__ __forceinline__ void finish_stat(double s, const FwdParams& P, float& r, float& rho)
{
    if (STAT == STAT_MX) {
        // G = (1/K sum m^p)^(1/p); r~ = fl32(coef * G); rho~ = 1 / fl32(r~ + eps)
        // (division by a power of two is an exact scaling: same result, far fewer instructions)
        double mean = P.inv_count != 0.0 ? __dmul_rn(s, P.inv_count) : __ddiv_rn(s, (double)P.K);
        double G = P.p == 2 ? __dsqrt_rn(mean) : mean;
        r = __double2float_rn(__dmul_rn((double)P.coef, G));
        rho = recip_sat(__fadd_rn(r, P.eps));
    } else if (STAT == STAT_POSTROUND) {
        // xbar = mean of the power-of-two-rounded block absmaxes; r~ = f^-1(xbar); rho~ = 1 / fl32(r~ + eps)
        const double xbar = P.inv_count != 0.0 ? __dmul_rn(s, P.inv_count) : __ddiv_rn(s, (double)P.K);
        r = __double2float_rn(postround_estimate(xbar, P.pr_table));
        rho = recip_sat(__fadd_rn(r, P.eps));
    } else if (STAT == STAT_RMS) {
        // r = fl32(sqrt(mean x^2 + eps)); rho = 1 / r
        double ms = P.inv_count != 0.0 ? __dmul_rn(s, P.inv_count) : __ddiv_rn(s, (double)P.D);
        r = __double2float_rn(__dsqrt_rn(__dadd_rn(ms, (double)P.eps)));
        rho = recip_sat(r);
    } else {
        r = 1.0f;
        rho = 1.0f;
    }
}

// sum of one double per warp over the WPR warps of a row group, in a fixed order.  Barrier ids are
// compile-time constants so that a kernel reserves only the barriers it uses (a dynamic id makes the
// compiler reserve all 16, which caps the number of resident CTAs).
template <int WPR>
__device__ __forceinline__ double group_sum(double v, int group, int w, double* smem)
{
    v = warp_sum(v);
    if (WPR > 1) {
        if ((threadIdx.x & 31) == 0) smem[group * WPR + w] = v;
        if (rows_per_cta(WPR) == 1) {
            __syncthreads();
        } else {
            switch (group) {
                case 0: group_barrier_id<1>(WPR * kWarp); break;
                case 1: group_barrier_id<2>(WPR * kWarp); break;
                case 2: group_barrier_id<3>(WPR * kWarp); break;
                default: group_barrier_id<4>(WPR * kWarp); break;
            }
        }
        double t = smem[group * WPR];
#pragma unroll
        for (int i = 1; i < WPR; ++i) t = __dadd_rn(t, smem[group * WPR + i]);
        v = t;
    }
    return v;
}

// ---- per-row work -------------------------------------------------------------------------------
// Lane `lane` of pass i of warp w owns piece k = (i*wpr + w)*32 + lane of the row: B contiguous elements,
// held in xr[i][] as packed pairs (zeros when k >= P.chunks).  A block of the format is LPB adjacent
// pieces (LPB = 1: the piece is the block).

// phase 1: block absmaxes m[i] (exact) and this lane's share of the row statistic
template <int B, int NPASS, int STAT, int LPB = 1>
__device__ __forceinline__ double block_stats(const uint32_t (&xr)[NPASS][B / 2], float (&m)[NPASS], int p, int lane = 0)
{
    constexpr int W = B / 2;
    double stat = 0.0;
    float2 ssa = make_float2(0.f, 0.f), ssb = make_float2(0.f, 0.f);   // four binary32 partial sums of squares
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        uint32_t m2 = absmax_bf16x2(xr[i][0], xr[i][1]);
#pragma unroll
        for (int j = 2; j < W; ++j) m2 = absmax_bf16x2(m2, xr[i][j]);
        m[i] = hmax_abs_to_f32(m2);
#pragma unroll
        for (int o = 1; o < LPB; o <<= 1) m[i] = fmaxf(m[i], __shfl_xor_sync(0xFFFFFFFFu, m[i], o));   // block absmax in every lane of the block
        const float mc = (LPB == 1 || (lane & (LPB - 1)) == 0) ? m[i] : 0.0f;   // each block counted once (adding 0 is exact)
        if (STAT == STAT_MX) {
            double md = (double)mc;
            stat = p == 2 ? __fma_rn(md, md, stat) : __dadd_rn(stat, md);   // m^2 is exact in binary64
        }
        if (STAT == STAT_POSTROUND) {   // 2^floor(log2 m): the absmax with its significand cleared (0 stays 0)
            const uint32_t u = __float_as_uint(mc);
            const uint32_t p2 = u >= 0x00800000u ? (u & 0x7F800000u) : (u != 0u ? 0x80000000u >> __clz(u) : 0u);   // subnormal: its leading bit
            stat = __dadd_rn(stat, (double)__uint_as_float(p2));
        }
        if (STAT == STAT_RMS) {
#pragma unroll
            for (int j = 0; j < W; j += 2) {
                const float2 a = bf16x2_to_f32x2(xr[i][j]), b = bf16x2_to_f32x2(xr[i][j + 1]);
                ssa = __ffma2_rn(a, a, ssa);
                ssb = __ffma2_rn(b, b, ssb);
            }
        }
    }
    if (STAT == STAT_RMS) stat = (double)ssa.x + (double)ssa.y + ((double)ssb.x + (double)ssb.y);
    return stat;
}

// Makes the compiler forget what it knows about the packed row: without this it keeps the binary32
// copies it unpacked for the sum of squares alive until the quantise phase (twice the registers).
template <int NPASS, int W>
__device__ __forceinline__ void forget_unpacked(uint32_t (&xr)[NPASS][W])
{
#pragma unroll
    for (int i = 0; i < NPASS; ++i)
#pragma unroll
        for (int j = 0; j < W; ++j) asm volatile("" : "+r"(xr[i][j]));
}

// byte offset of the scale of this lane's first block (pass 0) and the distance between passes
template <int WPR, int LPB = 1>
__device__ __forceinline__ void scale_addressing(const FwdParams& P, int64_t row, int w, int lane, int64_t& off0, int64_t& step)
{
    static_assert((kWarp / LPB) % 4 == 0, "a pass of one warp must cover whole groups of four scales");
    const int k0 = (w * kWarp + lane) / LPB;
    if (P.layout == MXN_SCALES_ROWMAJOR) {
        off0 = row * P.K + k0;
        step = WPR * (kWarp / LPB);
    } else {
        const int rr = (int)(row & 127);
        off0 = ((row >> 7) * P.tiles_per_row + (k0 >> 2)) * 512 + (rr & 31) * 16 + (rr >> 5) * 4 + (k0 & 3);
        step = (int64_t)WPR * (kWarp / LPB / 4) * 512;   // 32*WPR/LPB blocks further = that many / 4 tiles of 512 bytes
    }
}

// ---- one piece (B contiguous elements of one lane), given the row's rho ----------------------------------------
// E4M3 / E5M2 codes with an E8M0 scale, the paper's rounding rule or P.round: returns the scale byte, out[] = the codes.
// The __all_sync inside makes the choice between the one-product and the two-product form warp-uniform, so every lane
// of the warp must call this (inactive lanes with zero data).
template <int B, bool PAPER, int ELEM>
__device__ __forceinline__ uint32_t quantise_piece_fp8(const uint32_t (&x)[B / 2], float m, float rho, bool rho_normal, bool active,
                                                       int round, uint32_t (&out)[B / 4])
{
    constexpr int W = B / 2;
    // a = fl32(m * rho) is also the absmax of fl32(x * rho): rounding is monotone
    const float a = __fmul_rn(m, rho);
    const uint32_t sb = PAPER ? e8m0_scale_rceil_pow2<ELEM == 2 ? 15 : 8>(a) : e8m0_scale(a, round);
    const float inv = inv_scale(sb);
    // q = fl32(x*rho) * 2^(127-sb).  When neither factor product leaves the normal range the
    // two roundings collapse into the single product x * (rho * 2^(127-sb)).
    const float f = __fmul_rn(rho, inv);
    const bool fast = sb >= 16u && rho_normal && is_normal_f32(f);
    if (__all_sync(0xFFFFFFFFu, fast || !active)) {
        const float2 ff = make_float2(f, f);
#pragma unroll
        for (int j = 0; j < W; j += 2) {
            const float2 q0 = mul2(bf16x2_to_f32x2(x[j]), ff), q1 = mul2(bf16x2_to_f32x2(x[j + 1]), ff);
            out[j / 2] = cvt_fp8x4<ELEM>(q0.x, q0.y, q1.x, q1.y);
        }
    } else {
        const float2 rr = make_float2(rho, rho), ii = make_float2(inv, inv);
#pragma unroll
        for (int j = 0; j < W; j += 2) {
            const float2 q0 = mul2(mul2(bf16x2_to_f32x2(x[j]), rr), ii);
            const float2 q1 = mul2(mul2(bf16x2_to_f32x2(x[j + 1]), rr), ii);
            out[j / 2] = cvt_fp8x4<ELEM>(q0.x, q0.y, q1.x, q1.y);
        }
    }
    return sb;
}

// MXFP4: E2M1 codes two per byte with an E8M0 scale, S = 2^(ceil(log2 a) - 2) (4 = 2^2 is the largest power of two of E2M1)
template <int B>
__device__ __forceinline__ uint32_t quantise_piece_mxfp4(const uint32_t (&x)[B / 2], float m, float rho, bool rho_normal, bool active,
                                                         uint32_t (&out)[B / 8])
{
    constexpr int W = B / 2;
    const float a = __fmul_rn(m, rho);
    const uint32_t u = __float_as_uint(a), E = u >> 23;
    uint32_t sb;
    if (E >= 255u) sb = (u & 0x7FFFFFu) ? 0u : 254u;   // not finite (outside the contract)
    else sb = (uint32_t)max((int)E + ((u & 0x7FFFFFu) != 0u) - 2, 0);
    const float inv = inv_scale(sb);
    const float f = __fmul_rn(rho, inv);
    const bool fast = sb >= 16u && rho_normal && is_normal_f32(f);   // same argument as for E4M3
    if (__all_sync(0xFFFFFFFFu, fast || !active)) {
        const float2 ff = make_float2(f, f);
#pragma unroll
        for (int j = 0; j < W; j += 4) {
            const float2 q0 = mul2(bf16x2_to_f32x2(x[j]), ff), q1 = mul2(bf16x2_to_f32x2(x[j + 1]), ff);
            const float2 q2 = mul2(bf16x2_to_f32x2(x[j + 2]), ff), q3 = mul2(bf16x2_to_f32x2(x[j + 3]), ff);
            out[j / 4] = cvt_e2m1x8(q0.x, q0.y, q1.x, q1.y, q2.x, q2.y, q3.x, q3.y);
        }
    } else {
        const float2 rr = make_float2(rho, rho), ii = make_float2(inv, inv);
#pragma unroll
        for (int j = 0; j < W; j += 4) {
            const float2 q0 = mul2(mul2(bf16x2_to_f32x2(x[j]), rr), ii), q1 = mul2(mul2(bf16x2_to_f32x2(x[j + 1]), rr), ii);
            const float2 q2 = mul2(mul2(bf16x2_to_f32x2(x[j + 2]), rr), ii), q3 = mul2(mul2(bf16x2_to_f32x2(x[j + 3]), rr), ii);
            out[j / 4] = cvt_e2m1x8(q0.x, q0.y, q1.x, q1.y, q2.x, q2.y, q3.x, q3.y);
        }
    }
    return sb;
}

// NVFP4: one block of 16 elements: E4M3 block scale = E4M3(fl32(fl32(a/6) * global_scale)), a = fl32(m * rho~);
// element factor = fl32(rho~ * global_scale) / scale (0 when the scale is 0, saturating).  rho_g = fl32(rho * global_scale);
// rcp_sig = RN(1/(1+j/8)) for j = lane % 8 (fetched from the lane that holds the needed one with a shuffle: a
// lane-dependent index into constant memory would be replayed once per distinct index).  Every lane of the warp must call.
__device__ __forceinline__ uint32_t quantise_piece_nvfp4(const uint32_t (&x)[8], float m, float rho, float rho_g, bool rho_g_in_window,
                                                         float rcp_sig, float global_scale, bool active, uint32_t (&out)[2])
{
    const float a = __fmul_rn(m, rho);
    // the common case first, without the IEEE division sequences and decided for the whole warp at once:
    // numerators inside the window of the exact shortcut and a normal E4M3 scale
    uint32_t sc = cvt_e4m3x2(__fmul_rn(div_by_known(a, 6.0f, 0x1.555556p-3f), global_scale), 0.0f) & 0xFFu;
    const bool common = in_division_window(a) && sc >= 8u && rho_g_in_window;
    float inv;
    if (__all_sync(0xFFFFFFFFu, common || !active)) {
        const float d = __uint_as_float((sc << 20) + (120u << 23));            // (8+mf) * 2^(ef-10)
        const float c = __fmul_rn(__shfl_sync(0xFFFFFFFFu, rcp_sig, (int)(sc & 7u)), __uint_as_float((134u - (sc >> 3)) << 23));
        inv = div_by_known(rho_g, d, c);
    } else {
        sc = cvt_e4m3x2(__fmul_rn(div_by_6(a), global_scale), 0.0f) & 0xFFu;
        const float d = e4m3_to_f32(sc);
        if (sc >= 8u && rho_g_in_window) inv = div_by_e4m3_normal(rho_g, sc, d);
        else inv = d == 0.0f ? 0.0f : fminf(__fdiv_rn(rho_g, d), 3.402823466e+38f);   // saturates like rho itself
    }
    const float2 ii = make_float2(inv, inv);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t* xw = &x[h * 4];
        const float2 q0 = mul2(bf16x2_to_f32x2(xw[0]), ii), q1 = mul2(bf16x2_to_f32x2(xw[1]), ii);
        const float2 q2 = mul2(bf16x2_to_f32x2(xw[2]), ii), q3 = mul2(bf16x2_to_f32x2(xw[3]), ii);
        out[h] = cvt_e2m1x8(q0.x, q0.y, q1.x, q1.y, q2.x, q2.y, q3.x, q3.y);
    }
    return sc;
}

// phase 2 (E4M3 codes, E8M0 scales): scales, codes and their stores for this lane's blocks.
// PAPER selects the paper's rounding rule at compile time (the common case); otherwise P.round decides.
template <int B, int NPASS, int WPR, bool GAIN, bool PAPER, int ELEM = 0, int LPB = 1>
__device__ __forceinline__ void quantise_store_e4m3(const uint32_t (&xr)[NPASS][B / 2], const float (&m)[NPASS], float rho,
                                                    const FwdParams& P, int64_t row, int w, int lane)
{
    constexpr int W = B / 2;
    const bool rho_normal = is_normal_f32(rho);
    uint8_t* cp0 = P.codes + row * P.D + (int64_t)(w * kWarp + lane) * B;
    int64_t soff, sstep;
    scale_addressing<WPR, LPB>(P, row, w, lane, soff, sstep);
    uint8_t* sp0 = P.scales + soff;
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        const int k = (i * WPR + w) * kWarp + lane;
        const bool active = k < P.chunks;
        uint32_t out[W / 2];
        uint32_t sb;
        if (!GAIN) {
            sb = quantise_piece_fp8<B, PAPER, ELEM>(xr[i], m[i], rho, rho_normal, active, P.round, out);
        } else {
            // y = fl32(fl32(x*rho) * gamma); scales and codes from y
            uint32_t gr[W];
            if (active) {
                const uint16_t* gp = P.gain + (int64_t)k * B;
#pragma unroll
                for (int v = 0; v < W / 8; ++v) {
                    const uint4 g0 = __ldg(reinterpret_cast<const uint4*>(gp + v * 16));
                    const uint4 g1 = __ldg(reinterpret_cast<const uint4*>(gp + v * 16 + 8));
                    gr[v * 8 + 0] = g0.x; gr[v * 8 + 1] = g0.y; gr[v * 8 + 2] = g0.z; gr[v * 8 + 3] = g0.w;
                    gr[v * 8 + 4] = g1.x; gr[v * 8 + 5] = g1.y; gr[v * 8 + 6] = g1.z; gr[v * 8 + 7] = g1.w;
                }
            } else {
#pragma unroll
                for (int j = 0; j < W; ++j) gr[j] = 0u;
            }
            // two elements per instruction (packed binary32 multiplies, each half an ordinary IEEE operation)
            const float2 rr = make_float2(rho, rho);
            // the block's products are kept between the maximum and the conversion (the lane's input words of this
            // block and the gain are dead by then)
            float2 y[W];
            float2 my2 = make_float2(0.0f, 0.0f);
#pragma unroll
            for (int j = 0; j < W; ++j) {
                y[j] = mul2(mul2(bf16x2_to_f32x2(xr[i][j]), rr), bf16x2_to_f32x2(gr[j]));
                my2.x = fmaxf(my2.x, fabsf(y[j].x));
                my2.y = fmaxf(my2.y, fabsf(y[j].y));
            }
            float my = fmaxf(my2.x, my2.y);
#pragma unroll
            for (int o = 1; o < LPB; o <<= 1) my = fmaxf(my, __shfl_xor_sync(0xFFFFFFFFu, my, o));
            sb = PAPER ? e8m0_scale_rceil_pow2<ELEM == 2 ? 15 : 8>(my) : e8m0_scale(my, P.round);
            const float inv = inv_scale(sb);
            const float2 ii = make_float2(inv, inv);
#pragma unroll
            for (int j = 0; j < W; j += 2) {
                const float2 qa = mul2(y[j], ii), qb = mul2(y[j + 1], ii);
                out[j / 2] = cvt_fp8x4<ELEM>(qa.x, qa.y, qb.x, qb.y);
            }
        }
        if (active) {
            uint8_t* cp = cp0 + (int64_t)i * (WPR * kWarp * B);
            if (B == 16) {
                st_v4(cp, out);
            } else {
#pragma unroll
                for (int v = 0; v < W / 16; ++v) st_v8(cp + v * 32, &out[v * 8]);
            }
            if (LPB == 1 || (lane & (LPB - 1)) == 0) sp0[i * sstep] = (uint8_t)sb;
        }
    }
}

// phase 2 (MXFP4: E2M1 codes two per byte, E8M0 scales; the paper's rounding rule with 4 = 2^2 as the
// largest power of two of the element format): S = 2^(ceil(log2 a) - 2)
template <int B, int NPASS, int WPR, int LPB = 1>
__device__ __forceinline__ void quantise_store_mxfp4(const uint32_t (&xr)[NPASS][B / 2], const float (&m)[NPASS], float rho,
                                                     const FwdParams& P, int64_t row, int w, int lane)
{
    constexpr int W = B / 2;
    const bool rho_normal = is_normal_f32(rho);
    uint8_t* cp0 = P.codes + row * (P.D / 2) + (int64_t)(w * kWarp + lane) * (B / 2);
    int64_t soff, sstep;
    scale_addressing<WPR, LPB>(P, row, w, lane, soff, sstep);
    uint8_t* sp0 = P.scales + soff;
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        const int k = (i * WPR + w) * kWarp + lane;
        const bool active = k < P.chunks;
        uint32_t out[W / 4];
        const uint32_t sb = quantise_piece_mxfp4<B>(xr[i], m[i], rho, rho_normal, active, out);
        if (active) {
            uint8_t* cp = cp0 + (int64_t)i * (WPR * kWarp * (B / 2));
            if (B == 16) st_v2(cp, out);
            else if (B == 32) st_v4(cp, out);
            else st_v8(cp, out);
            if (LPB == 1 || (lane & (LPB - 1)) == 0) sp0[i * sstep] = (uint8_t)sb;
        }
    }
}

// phase 2 (NVFP4): E4M3 block scales, E2M1 codes two per byte, B = 16
template <int NPASS, int WPR>
__device__ __forceinline__ void quantise_store_nvfp4(const uint32_t (&xr)[NPASS][8], const float (&m)[NPASS], float rho,
                                                     const FwdParams& P, int64_t row, int w, int lane)
{
    const float rho_g = __fmul_rn(rho, P.global_scale);
    const bool rho_g_in_window = in_division_window(rho_g);
    // RN(1/(1+j/8)), j = lane % 8, held one per lane and fetched with a shuffle: a lane-dependent index into
    // constant memory would be replayed once per distinct index
    const float rcp_sig = kRcpE4M3Significand[lane & 7];
    uint8_t* cp0 = P.codes + row * (P.D / 2) + (int64_t)(w * kWarp + lane) * 8;
    int64_t soff, sstep;
    scale_addressing<WPR>(P, row, w, lane, soff, sstep);
    uint8_t* sp0 = P.scales + soff;
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        const int k = (i * WPR + w) * kWarp + lane;
        uint32_t out[2];
        const uint32_t sc = quantise_piece_nvfp4(xr[i], m[i], rho, rho_g, rho_g_in_window, rcp_sig, P.global_scale, k < P.K, out);
        if (k < P.K) {
            st_v2(cp0 + (int64_t)i * (WPR * kWarp * 8), out);
            sp0[i * sstep] = (uint8_t)sc;
        }
    }
}

// NVFP4 with a lane owning two adjacent blocks (32 contiguous elements): the per-block scalar arithmetic of the two
// blocks runs as packed binary32 pairs (each half an ordinary IEEE operation, so results are those of
// quantise_piece_nvfp4 bit for bit), both E4M3 scale bytes come out of one conversion and leave as one 16-bit store,
// and the 32 codes leave as one 16-byte store.  Every lane of the warp must call.
__device__ __forceinline__ float2 div2_by_known(float2 a, float2 d, float2 c)
{
    const float2 q = __fmul2_rn(a, c);
    const float2 r = __ffma2_rn(make_float2(-d.x, -d.y), q, a);
    return __ffma2_rn(r, c, q);
}
__device__ __forceinline__ uint32_t quantise_pair_nvfp4(const uint32_t (&x)[16], float m0, float m1, float rho, float rho_g,
                                                        bool rho_g_in_window, float rcp_sig, float global_scale, bool active,
                                                        uint32_t (&out)[4])
{
    const float2 a = __fmul2_rn(make_float2(m0, m1), make_float2(rho, rho));
    const float2 six = make_float2(6.0f, 6.0f), c6 = make_float2(0x1.555556p-3f, 0x1.555556p-3f), gs = make_float2(global_scale, global_scale);
    const float2 t = __fmul2_rn(div2_by_known(a, six, c6), gs);
    uint32_t sc2 = cvt_e4m3x2(t.x, t.y);                 // block 0 in the low byte
    uint32_t sc0 = sc2 & 0xFFu, sc1 = sc2 >> 8;
    const bool common = in_division_window(a.x) && in_division_window(a.y) && sc0 >= 8u && sc1 >= 8u && rho_g_in_window;
    float2 inv;
    if (__all_sync(0xFFFFFFFFu, common || !active)) {
        const float2 d = make_float2(__uint_as_float((sc0 << 20) + (120u << 23)), __uint_as_float((sc1 << 20) + (120u << 23)));
        const float2 c = make_float2(
            __fmul_rn(__shfl_sync(0xFFFFFFFFu, rcp_sig, (int)(sc0 & 7u)), __uint_as_float((134u - (sc0 >> 3)) << 23)),
            __fmul_rn(__shfl_sync(0xFFFFFFFFu, rcp_sig, (int)(sc1 & 7u)), __uint_as_float((134u - (sc1 >> 3)) << 23)));
        inv = div2_by_known(make_float2(rho_g, rho_g), d, c);
    } else {
        float iv[2];
        uint32_t sc[2];
        const float av[2] = {a.x, a.y};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            sc[h] = cvt_e4m3x2(__fmul_rn(div_by_6(av[h]), global_scale), 0.0f) & 0xFFu;
            const float d = e4m3_to_f32(sc[h]);
            if (sc[h] >= 8u && rho_g_in_window) iv[h] = div_by_e4m3_normal(rho_g, sc[h], d);
            else iv[h] = d == 0.0f ? 0.0f : fminf(__fdiv_rn(rho_g, d), 3.402823466e+38f);
        }
        sc0 = sc[0];
        sc1 = sc[1];
        sc2 = sc0 | (sc1 << 8);
        inv = make_float2(iv[0], iv[1]);
    }
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        const float f = h < 2 ? inv.x : inv.y;
        const float2 ii = make_float2(f, f);
        const uint32_t* xw = &x[h * 4];
        const float2 q0 = mul2(bf16x2_to_f32x2(xw[0]), ii), q1 = mul2(bf16x2_to_f32x2(xw[1]), ii);
        const float2 q2 = mul2(bf16x2_to_f32x2(xw[2]), ii), q3 = mul2(bf16x2_to_f32x2(xw[3]), ii);
        out[h] = cvt_e2m1x8(q0.x, q0.y, q1.x, q1.y, q2.x, q2.y, q3.x, q3.y);
    }
    return sc2;
}

// phase 2 of the pair kernel: lane `lane` of pass i of warp w owns blocks 2k and 2k+1, k = (i*WPR + w)*32 + lane
template <int NPASS, int WPR>
__device__ __forceinline__ void quantise_store_nvfp4_pair(const uint32_t (&xr)[NPASS][16], const float (&m0)[NPASS], const float (&m1)[NPASS],
                                                          float rho, const FwdParams& P, int64_t row, int w, int lane)
{
    const float rho_g = __fmul_rn(rho, P.global_scale);
    const bool rho_g_in_window = in_division_window(rho_g);
    const float rcp_sig = kRcpE4M3Significand[lane & 7];
    uint8_t* cp0 = P.codes + row * (P.D / 2) + (int64_t)(w * kWarp + lane) * 16;
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        const int k = (i * WPR + w) * kWarp + lane;
        const bool active = k < P.chunks;
        uint32_t out[4];
        const uint32_t sc2 = quantise_pair_nvfp4(xr[i], m0[i], m1[i], rho, rho_g, rho_g_in_window, rcp_sig, P.global_scale, active, out);
        if (active) {
            st_v4(cp0 + (int64_t)i * (WPR * kWarp * 16), out);
            const int kb = 2 * k;
            int64_t off;
            if (P.layout == MXN_SCALES_ROWMAJOR) {
                off = row * P.K + kb;
            } else {
                const int rr = (int)(row & 127);
                off = ((row >> 7) * P.tiles_per_row + (kb >> 2)) * 512 + (rr & 31) * 16 + (rr >> 5) * 4 + (kb & 3);
            }
            *reinterpret_cast<uint16_t*>(P.scales + off) = (uint16_t)sc2;      // two adjacent scale bytes (off is even)
        }
    }
}

}  // namespace mxn
#endif  // MXN_ROW_CUH_
