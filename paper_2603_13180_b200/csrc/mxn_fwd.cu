// Forward kernels: MXCast, fused RMSNorm+MXCast (Algorithm 1), MXNorm (Algorithm 2) and its post-round
// ablation with E4M3 codes / E8M0 scales; the MXFP4 (E2M1 / E8M0), NVFP4 (E2M1 / E4M3 scales) and
// E5M2 variants.
//
// Work decomposition (memory-bound streaming map with one scalar reduction per row):
//   * a row is handled by a "row group" of WPR warps (2 for D = 4096 at B = 32: at most 64 elements
//     per lane) and stays in registers between the statistics phase and the quantise phase - every
//     input byte is read from HBM exactly once, with 32-byte loads that bypass L1;
//   * one lane owns one whole block per pass (B contiguous elements = 2B bytes), so the block
//     absmax needs no cross-lane traffic, the scale is computed once per block, a warp writes
//     32 consecutive scale bytes and 32*B consecutive code bytes per pass (B = 64: two adjacent lanes
//     own the halves of a block - LPB = 2 "lanes per block" - and exchange their maxima with one shuffle,
//     which keeps a lane at 32 contiguous elements per pass and the per-lane code identical to B = 32);
//   * the only cross-lane step is the row statistic: K = D/B block values (MXNorm) instead of
//     D squares (RMSNorm), reduced in binary64 by shuffles (and through shared memory when a row
//     spans several warps);
//   * short-lived CTAs (one per 1-4 rows), launched with programmatic stream serialisation: measured
//     faster on B200 than resident CTAs, with or without TMA staging.
#include <cmath>
#include <mutex>

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

// ---- post-round estimator tables (appendix "Post-round MXNorm") ------------------------------------
// f^-1 sampled at the 65 nodes 2^(i/64) of [1,2] for each block size, with the slope of every interval;
// filled by postround_prepare() on the host, read by finish_stat<STAT_POSTROUND>.
constexpr int kPrIntervals = 64;
__device__ __constant__ double c_pr_nodes[kPrIntervals + 1];
__device__ __constant__ double c_pr_values[3][kPrIntervals + 1];
__device__ __constant__ double c_pr_slopes[3][kPrIntervals];

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
        float den = __fadd_rn(r, P.eps);
        rho = den == 0.0f ? 0.0f : __fdiv_rn(1.0f, den);
    } else if (STAT == STAT_POSTROUND) {
        // xbar = mean of the power-of-two-rounded block absmaxes; r~ = f^-1(xbar); rho~ = 1 / fl32(r~ + eps)
        const double xbar = P.inv_count != 0.0 ? __dmul_rn(s, P.inv_count) : __ddiv_rn(s, (double)P.K);
        r = __double2float_rn(postround_estimate(xbar, P.pr_table));
        float den = __fadd_rn(r, P.eps);
        rho = den == 0.0f ? 0.0f : __fdiv_rn(1.0f, den);
    } else if (STAT == STAT_RMS) {
        // r = fl32(sqrt(mean x^2 + eps)); rho = 1 / r
        double ms = P.inv_count != 0.0 ? __dmul_rn(s, P.inv_count) : __ddiv_rn(s, (double)P.D);
        r = __double2float_rn(__dsqrt_rn(__dadd_rn(ms, (double)P.eps)));
        rho = r == 0.0f ? 0.0f : __fdiv_rn(1.0f, r);
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
        if (STAT == STAT_POSTROUND)   // 2^floor(log2 m): the absmax with its significand cleared (0 stays 0)
            stat = __dadd_rn(stat, (double)__uint_as_float(__float_as_uint(mc) & 0x7F800000u));
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
            // a = fl32(m * rho) is also the absmax of fl32(x * rho): rounding is monotone
            const float a = __fmul_rn(m[i], rho);
            sb = PAPER ? e8m0_scale_rceil_pow2<ELEM == 2 ? 15 : 8>(a) : e8m0_scale(a, P.round);
            const float inv = inv_scale(sb);
            // q = fl32(x*rho) * 2^(127-sb).  When neither factor product leaves the normal range the
            // two roundings collapse into the single product x * (rho * 2^(127-sb)).
            const float f = __fmul_rn(rho, inv);
            const bool fast = sb >= 16u && rho_normal && is_normal_f32(f);
            if (__all_sync(0xFFFFFFFFu, fast || !active)) {
                const float2 ff = make_float2(f, f);
#pragma unroll
                for (int j = 0; j < W; j += 2) {
                    const float2 q0 = mul2(bf16x2_to_f32x2(xr[i][j]), ff), q1 = mul2(bf16x2_to_f32x2(xr[i][j + 1]), ff);
                    out[j / 2] = cvt_fp8x4<ELEM>(q0.x, q0.y, q1.x, q1.y);
                }
            } else {
                const float2 rr = make_float2(rho, rho), ii = make_float2(inv, inv);
#pragma unroll
                for (int j = 0; j < W; j += 2) {
                    const float2 q0 = mul2(mul2(bf16x2_to_f32x2(xr[i][j]), rr), ii);
                    const float2 q1 = mul2(mul2(bf16x2_to_f32x2(xr[i][j + 1]), rr), ii);
                    out[j / 2] = cvt_fp8x4<ELEM>(q0.x, q0.y, q1.x, q1.y);
                }
            }
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
            float my = 0.0f;
#pragma unroll
            for (int j = 0; j < W; ++j) {
                const float y0 = __fmul_rn(__fmul_rn(bf16_lo(xr[i][j]), rho), bf16_lo(gr[j]));
                const float y1 = __fmul_rn(__fmul_rn(bf16_hi(xr[i][j]), rho), bf16_hi(gr[j]));
                my = fmaxf(my, fmaxf(fabsf(y0), fabsf(y1)));
            }
#pragma unroll
            for (int o = 1; o < LPB; o <<= 1) my = fmaxf(my, __shfl_xor_sync(0xFFFFFFFFu, my, o));
            sb = PAPER ? e8m0_scale_rceil_pow2<ELEM == 2 ? 15 : 8>(my) : e8m0_scale(my, P.round);
            const float inv = inv_scale(sb);
#pragma unroll
            for (int j = 0; j < W; j += 2) {
                const float y0 = __fmul_rn(__fmul_rn(bf16_lo(xr[i][j]), rho), bf16_lo(gr[j]));
                const float y1 = __fmul_rn(__fmul_rn(bf16_hi(xr[i][j]), rho), bf16_hi(gr[j]));
                const float y2 = __fmul_rn(__fmul_rn(bf16_lo(xr[i][j + 1]), rho), bf16_lo(gr[j + 1]));
                const float y3 = __fmul_rn(__fmul_rn(bf16_hi(xr[i][j + 1]), rho), bf16_hi(gr[j + 1]));
                out[j / 2] = cvt_fp8x4<ELEM>(__fmul_rn(y0, inv), __fmul_rn(y1, inv), __fmul_rn(y2, inv), __fmul_rn(y3, inv));
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
        const float a = __fmul_rn(m[i], rho);
        const uint32_t u = __float_as_uint(a), E = u >> 23;
        uint32_t sb;
        if (E >= 255u) sb = (u & 0x7FFFFFu) ? 0u : 254u;   // not finite (outside the contract)
        else sb = (uint32_t)max((int)E + ((u & 0x7FFFFFu) != 0u) - 2, 0);
        const float inv = inv_scale(sb);
        const float f = __fmul_rn(rho, inv);
        const bool fast = sb >= 16u && rho_normal && is_normal_f32(f);   // same argument as for E4M3
        uint32_t out[W / 4];
        if (__all_sync(0xFFFFFFFFu, fast || !active)) {
            const float2 ff = make_float2(f, f);
#pragma unroll
            for (int j = 0; j < W; j += 4) {
                const float2 q0 = mul2(bf16x2_to_f32x2(xr[i][j]), ff), q1 = mul2(bf16x2_to_f32x2(xr[i][j + 1]), ff);
                const float2 q2 = mul2(bf16x2_to_f32x2(xr[i][j + 2]), ff), q3 = mul2(bf16x2_to_f32x2(xr[i][j + 3]), ff);
                out[j / 4] = cvt_e2m1x8(q0.x, q0.y, q1.x, q1.y, q2.x, q2.y, q3.x, q3.y);
            }
        } else {
            const float2 rr = make_float2(rho, rho), ii = make_float2(inv, inv);
#pragma unroll
            for (int j = 0; j < W; j += 4) {
                const float2 q0 = mul2(mul2(bf16x2_to_f32x2(xr[i][j]), rr), ii), q1 = mul2(mul2(bf16x2_to_f32x2(xr[i][j + 1]), rr), ii);
                const float2 q2 = mul2(mul2(bf16x2_to_f32x2(xr[i][j + 2]), rr), ii), q3 = mul2(mul2(bf16x2_to_f32x2(xr[i][j + 3]), rr), ii);
                out[j / 4] = cvt_e2m1x8(q0.x, q0.y, q1.x, q1.y, q2.x, q2.y, q3.x, q3.y);
            }
        }
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
        // block scale = E4M3(fl32(fl32(a/6) * global_scale)), a = fl32(m * rho~);
        // element factor = fl32(rho~ * global_scale) / scale (0 when the scale is 0)
        const float a = __fmul_rn(m[i], rho);
        // the common case first, without the IEEE division sequences and decided for the whole warp at once:
        // numerators inside the window of the exact shortcut and a normal E4M3 scale
        uint32_t sc = cvt_e4m3x2(__fmul_rn(div_by_known(a, 6.0f, 0x1.555556p-3f), P.global_scale), 0.0f) & 0xFFu;
        const bool common = in_division_window(a) && sc >= 8u && rho_g_in_window;
        float inv;
        if (__all_sync(0xFFFFFFFFu, common || k >= P.K)) {
            const float d = __uint_as_float((sc << 20) + (120u << 23));            // (8+mf) * 2^(ef-10)
            const float c = __fmul_rn(__shfl_sync(0xFFFFFFFFu, rcp_sig, (int)(sc & 7u)), __uint_as_float((134u - (sc >> 3)) << 23));
            inv = div_by_known(rho_g, d, c);
        } else {
            sc = cvt_e4m3x2(__fmul_rn(div_by_6(a), P.global_scale), 0.0f) & 0xFFu;
            const float d = e4m3_to_f32(sc);
            if (sc >= 8u && rho_g_in_window) inv = div_by_e4m3_normal(rho_g, sc, d);
            else inv = d == 0.0f ? 0.0f : __fdiv_rn(rho_g, d);
        }
        uint32_t out[2];
        const float2 ii = make_float2(inv, inv);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t* xw = &xr[i][h * 4];
            const float2 q0 = mul2(bf16x2_to_f32x2(xw[0]), ii), q1 = mul2(bf16x2_to_f32x2(xw[1]), ii);
            const float2 q2 = mul2(bf16x2_to_f32x2(xw[2]), ii), q3 = mul2(bf16x2_to_f32x2(xw[3]), ii);
            out[h] = cvt_e2m1x8(q0.x, q0.y, q1.x, q1.y, q2.x, q2.y, q3.x, q3.y);
        }
        if (k < P.K) {
            st_v2(cp0 + (int64_t)i * (WPR * kWarp * 8), out);
            sp0[i * sstep] = (uint8_t)sc;
        }
    }
}

// ---- register-direct kernels: one row per row group, loaded straight from global memory -----------
// Generic path: any D % B == 0, rows spanning up to 8 warps, optional gain.
template <int B, int NPASS, bool COHERENT = false>
__device__ __forceinline__ void load_row_direct(uint32_t (&xr)[NPASS][B / 2], const uint16_t* xrow, int K, int wpr, int w, int lane)
{
    constexpr int W = B / 2;
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        const int k = (i * wpr + w) * kWarp + lane;
        if (k < K) {
            const uint16_t* p = xrow + (int64_t)k * B;
#pragma unroll
            for (int v = 0; v < W / 8; ++v) {
                if (COHERENT) ld_v8_coherent(p + v * 16, &xr[i][v * 8]);
                else ld_v8(p + v * 16, &xr[i][v * 8]);
            }
        } else {
#pragma unroll
            for (int j = 0; j < W; ++j) xr[i][j] = 0u;
        }
    }
}

template <int B, int NPASS, int WPR, int STAT, bool GAIN, bool PAPER, int LPB = 1>
__global__ void __launch_bounds__(cta_warps(WPR) * 32, MXN_FWD_MIN_CTAS) fwd_e4m3_kernel(const FwdParams P)
{
    __shared__ double red[WPR > 1 ? cta_warps(WPR) : 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int group = warp / WPR, w = warp - group * WPR;
    const int64_t row = (int64_t)blockIdx.x * rows_per_cta(WPR) + group;
    pdl_prologue();
    if (row >= P.T) return;   // whole row group leaves together

    uint32_t xr[NPASS][B / 2];
    float m[NPASS];
    load_row_direct<B, NPASS>(xr, P.x + row * P.D, P.chunks, WPR, w, lane);
    double stat = block_stats<B, NPASS, STAT, LPB>(xr, m, P.p, lane);
    if (STAT == STAT_RMS) forget_unpacked<NPASS, B / 2>(xr);
    float r = 1.0f, rho = 1.0f;
    if (STAT != STAT_NONE) {
        stat = group_sum<WPR>(stat, group, w, red);
        finish_stat<STAT>(stat, P, r, rho);
        if (P.rms_out != nullptr && w == 0 && lane == 0) P.rms_out[row] = r;
    }
    quantise_store_e4m3<B, NPASS, WPR, GAIN, PAPER, 0, LPB>(xr, m, rho, P, row, w, lane);
}

// Residual add fused in front of MXNorm: h = bf16(x + res) is written out as the new residual stream and
// normalised from registers (reads 4D bytes, writes 2D + D + D/B per row instead of two passes over h).
__device__ __forceinline__ uint32_t add_bf16x2(uint32_t a, uint32_t b)
{
    // each half: binary32 sum of two exactly widened bf16 values, rounded once to bf16 (RN-even)
    const float lo = __fadd_rn(bf16_lo(a), bf16_lo(b)), hi = __fadd_rn(bf16_hi(a), bf16_hi(b));
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

template <int B, int NPASS, int WPR, int LPB = 1>
__global__ void __launch_bounds__(cta_warps(WPR) * 32, MXN_FWD_MIN_CTAS) fwd_add_mx_kernel(const FwdParams P)
{
    constexpr int W = B / 2;
    __shared__ double red[WPR > 1 ? cta_warps(WPR) : 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int group = warp / WPR, w = warp - group * WPR;
    const int64_t row = (int64_t)blockIdx.x * rows_per_cta(WPR) + group;
    pdl_prologue();
    if (row >= P.T) return;

    uint32_t xr[NPASS][W];
    float m[NPASS];
    load_row_direct<B, NPASS, true>(xr, P.x + row * P.D, P.chunks, WPR, w, lane);   // h_out may alias x or residual
    {
        uint32_t rr[NPASS][W];
        load_row_direct<B, NPASS, true>(rr, P.residual + row * P.D, P.chunks, WPR, w, lane);
        uint16_t* hrow = P.h_out + row * P.D;
#pragma unroll
        for (int i = 0; i < NPASS; ++i) {
#pragma unroll
            for (int j = 0; j < W; ++j) xr[i][j] = add_bf16x2(xr[i][j], rr[i][j]);
            const int k = (i * WPR + w) * kWarp + lane;
            if (k < P.chunks) {
#pragma unroll
                for (int v = 0; v < W / 8; ++v) st_v8(hrow + (int64_t)k * B + v * 16, &xr[i][v * 8]);
            }
        }
    }
    double stat = block_stats<B, NPASS, STAT_MX, LPB>(xr, m, P.p, lane);
    stat = group_sum<WPR>(stat, group, w, red);
    float r, rho;
    finish_stat<STAT_MX>(stat, P, r, rho);
    if (P.rms_out != nullptr && w == 0 && lane == 0) P.rms_out[row] = r;
    quantise_store_e4m3<B, NPASS, WPR, false, true, 0, LPB>(xr, m, rho, P, row, w, lane);
}

// plain MXCast to E5M2 codes (gradient tensors), the paper's rounding rule with 2^15
template <int B, int NPASS, int WPR, int LPB = 1>
__global__ void __launch_bounds__(cta_warps(WPR) * 32, MXN_FWD_MIN_CTAS) cast_e5m2_kernel(const FwdParams P)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int group = warp / WPR, w = warp - group * WPR;
    const int64_t row = (int64_t)blockIdx.x * rows_per_cta(WPR) + group;
    pdl_prologue();
    if (row >= P.T) return;
    uint32_t xr[NPASS][B / 2];
    float m[NPASS];
    load_row_direct<B, NPASS>(xr, P.x + row * P.D, P.chunks, WPR, w, lane);
    (void)block_stats<B, NPASS, STAT_NONE, LPB>(xr, m, 2, lane);
    quantise_store_e4m3<B, NPASS, WPR, false, true, 2, LPB>(xr, m, 1.0f, P, row, w, lane);
}

// E2M1 codes with E8M0 scales (MXFP4): no gain, the paper's rounding rule
template <int B, int NPASS, int WPR, int STAT, int LPB = 1>
__global__ void __launch_bounds__(cta_warps(WPR) * 32, MXN_FWD_MIN_CTAS) fwd_mxfp4_kernel(const FwdParams P)
{
    __shared__ double red[WPR > 1 ? cta_warps(WPR) : 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int group = warp / WPR, w = warp - group * WPR;
    const int64_t row = (int64_t)blockIdx.x * rows_per_cta(WPR) + group;
    pdl_prologue();
    if (row >= P.T) return;

    uint32_t xr[NPASS][B / 2];
    float m[NPASS];
    load_row_direct<B, NPASS>(xr, P.x + row * P.D, P.chunks, WPR, w, lane);
    double stat = block_stats<B, NPASS, STAT, LPB>(xr, m, P.p, lane);
    if (STAT == STAT_RMS) forget_unpacked<NPASS, B / 2>(xr);
    float r = 1.0f, rho = 1.0f;
    if (STAT != STAT_NONE) {
        stat = group_sum<WPR>(stat, group, w, red);
        finish_stat<STAT>(stat, P, r, rho);
        if (P.rms_out != nullptr && w == 0 && lane == 0) P.rms_out[row] = r;
    }
    quantise_store_mxfp4<B, NPASS, WPR, LPB>(xr, m, rho, P, row, w, lane);
}

template <int NPASS, int WPR, int STAT>
__global__ void __launch_bounds__(cta_warps(WPR) * 32, MXN_FWD_MIN_CTAS) fwd_nvfp4_kernel(const FwdParams P)
{
    __shared__ double red[WPR > 1 ? cta_warps(WPR) : 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int group = warp / WPR, w = warp - group * WPR;
    const int64_t row = (int64_t)blockIdx.x * rows_per_cta(WPR) + group;
    pdl_prologue();
    if (row >= P.T) return;

    uint32_t xr[NPASS][8];
    float m[NPASS];
    load_row_direct<16, NPASS>(xr, P.x + row * P.D, P.chunks, WPR, w, lane);
    double stat = block_stats<16, NPASS, STAT>(xr, m, P.p);
    if (STAT == STAT_RMS) forget_unpacked<NPASS, 8>(xr);
    stat = group_sum<WPR>(stat, group, w, red);
    float r, rho;
    finish_stat<STAT>(stat, P, r, rho);
    if (P.rms_out != nullptr && w == 0 && lane == 0) P.rms_out[row] = r;
    quantise_store_nvfp4<NPASS, WPR>(xr, m, rho, P, row, w, lane);
}

// ---- dispatch ---------------------------------------------------------------------------------
typedef void (*fwd_fn)(const FwdParams);

// In the templates below B is the number of elements a lane holds per pass and LPB the lanes per block
// (block size of the format = B * LPB: 16 = 16x1, 32 = 32x1, 64 = 32x2).
// The headline kernels (E4M3 codes or NVFP4, no gain, the paper's rounding rule) exist for every number of
// warps per row in kFineWpr, so that hidden sizes of the form {3,5,7} * 2^r fill their lanes; the
// other variants exist for power-of-two warps per row only.
static const int kFineWpr[] = {1, 2, 3, 4, 5, 6, 7, 8, 16};
static const int kCoarseWpr[] = {1, 2, 4, 8, 16};

template <int B, int LPB, int NPASS, int STAT, bool GAIN, bool PAPER, bool FINE>
static fwd_fn e4m3_by_wpr(int wpr)
{
    switch (wpr) {
        case 1: return fwd_e4m3_kernel<B, NPASS, 1, STAT, GAIN, PAPER, LPB>;
        case 2: return fwd_e4m3_kernel<B, NPASS, 2, STAT, GAIN, PAPER, LPB>;
        case 4: return fwd_e4m3_kernel<B, NPASS, 4, STAT, GAIN, PAPER, LPB>;
        case 8: return fwd_e4m3_kernel<B, NPASS, 8, STAT, GAIN, PAPER, LPB>;
        case 16: return fwd_e4m3_kernel<B, NPASS, 16, STAT, GAIN, PAPER, LPB>;
        default: break;
    }
    if constexpr (FINE) {
        switch (wpr) {
            case 3: return fwd_e4m3_kernel<B, NPASS, 3, STAT, GAIN, PAPER, LPB>;
            case 5: return fwd_e4m3_kernel<B, NPASS, 5, STAT, GAIN, PAPER, LPB>;
            case 6: return fwd_e4m3_kernel<B, NPASS, 6, STAT, GAIN, PAPER, LPB>;
            case 7: return fwd_e4m3_kernel<B, NPASS, 7, STAT, GAIN, PAPER, LPB>;
            default: break;
        }
    }
    return nullptr;
}

// Every variant exists for WPR = 1 with any pass count and for WPR > 1 with the full pass count; the FINE
// ones also for WPR > 1 with one pass and (four-pass kernels) with two.
template <int B, int LPB, int STAT, bool GAIN, bool PAPER>
static fwd_fn pick_e4m3(int wpr, int npass)
{
    constexpr int MAXP = MXN_FWD_MAX_ELEMS / B;
    constexpr bool FINE = !GAIN && PAPER && STAT != STAT_POSTROUND;
    if (wpr > 1) {
        if (npass == MAXP) return e4m3_by_wpr<B, LPB, MAXP, STAT, GAIN, PAPER, FINE>(wpr);
        if (FINE && MAXP >= 4 && npass == MAXP / 2) return e4m3_by_wpr<B, LPB, (MAXP >= 4 ? MAXP / 2 : 1), STAT, GAIN, PAPER, FINE>(wpr);
        if (FINE && npass == 1) return e4m3_by_wpr<B, LPB, 1, STAT, GAIN, PAPER, FINE>(wpr);
        return nullptr;
    }
    switch (npass) {
        case 1: return fwd_e4m3_kernel<B, 1, 1, STAT, GAIN, PAPER, LPB>;
        case 2: return fwd_e4m3_kernel<B, (MAXP >= 2 ? 2 : MAXP), 1, STAT, GAIN, PAPER, LPB>;
        case 3: return fwd_e4m3_kernel<B, (MAXP >= 3 ? 3 : MAXP), 1, STAT, GAIN, PAPER, LPB>;
        default: return fwd_e4m3_kernel<B, MAXP, 1, STAT, GAIN, PAPER, LPB>;
    }
}
template <int B, int LPB, bool PAPER>
static fwd_fn pick_stat(int stat, bool gain, int wpr, int npass)
{
    switch (stat) {
        case STAT_NONE: return pick_e4m3<B, LPB, STAT_NONE, false, PAPER>(wpr, npass);
        case STAT_RMS: return gain ? pick_e4m3<B, LPB, STAT_RMS, true, PAPER>(wpr, npass) : pick_e4m3<B, LPB, STAT_RMS, false, PAPER>(wpr, npass);
        case STAT_MX: return gain ? pick_e4m3<B, LPB, STAT_MX, true, PAPER>(wpr, npass) : pick_e4m3<B, LPB, STAT_MX, false, PAPER>(wpr, npass);
        case STAT_POSTROUND: return (gain || !PAPER) ? nullptr : pick_e4m3<B, LPB, STAT_POSTROUND, false, true>(wpr, npass);
        default: return nullptr;
    }
}
template <int B, int LPB>
static fwd_fn pick_round(int round, int stat, bool gain, int wpr, int npass)
{
    return round == MXN_ROUND_RCEIL_POW2 ? pick_stat<B, LPB, true>(stat, gain, wpr, npass) : pick_stat<B, LPB, false>(stat, gain, wpr, npass);
}
template <int B, int LPB, int STAT>
static fwd_fn pick_mxfp4(int wpr, int npass)
{
    constexpr int MAXP = MXN_FWD_MAX_ELEMS / B;
    if (wpr == 2) return fwd_mxfp4_kernel<B, MAXP, 2, STAT, LPB>;
    if (wpr == 4) return fwd_mxfp4_kernel<B, MAXP, 4, STAT, LPB>;
    if (wpr == 8) return fwd_mxfp4_kernel<B, MAXP, 8, STAT, LPB>;
    if (wpr == 16) return fwd_mxfp4_kernel<B, MAXP, 16, STAT, LPB>;
    if (wpr != 1) return nullptr;
    switch (npass) {
        case 1: return fwd_mxfp4_kernel<B, 1, 1, STAT, LPB>;
        case 2: return fwd_mxfp4_kernel<B, (MAXP >= 2 ? 2 : MAXP), 1, STAT, LPB>;
        case 3: return fwd_mxfp4_kernel<B, (MAXP >= 3 ? 3 : MAXP), 1, STAT, LPB>;
        default: return fwd_mxfp4_kernel<B, MAXP, 1, STAT, LPB>;
    }
}
template <int B, int LPB>
static fwd_fn pick_add_mx(int wpr, int npass)
{
    constexpr int MAXP = MXN_FWD_MAX_ELEMS / B;
    if (wpr == 2) return fwd_add_mx_kernel<B, MAXP, 2, LPB>;
    if (wpr == 4) return fwd_add_mx_kernel<B, MAXP, 4, LPB>;
    if (wpr == 8) return fwd_add_mx_kernel<B, MAXP, 8, LPB>;
    if (wpr == 16) return fwd_add_mx_kernel<B, MAXP, 16, LPB>;
    if (wpr != 1) return nullptr;
    switch (npass) {
        case 1: return fwd_add_mx_kernel<B, 1, 1, LPB>;
        case 2: return fwd_add_mx_kernel<B, (MAXP >= 2 ? 2 : MAXP), 1, LPB>;
        case 3: return fwd_add_mx_kernel<B, (MAXP >= 3 ? 3 : MAXP), 1, LPB>;
        default: return fwd_add_mx_kernel<B, MAXP, 1, LPB>;
    }
}

template <int B, int LPB>
static fwd_fn pick_e5m2(int wpr, int npass)
{
    constexpr int MAXP = MXN_FWD_MAX_ELEMS / B;
    if (wpr == 2) return cast_e5m2_kernel<B, MAXP, 2, LPB>;
    if (wpr == 4) return cast_e5m2_kernel<B, MAXP, 4, LPB>;
    if (wpr == 8) return cast_e5m2_kernel<B, MAXP, 8, LPB>;
    if (wpr == 16) return cast_e5m2_kernel<B, MAXP, 16, LPB>;
    if (wpr != 1) return nullptr;
    switch (npass) {
        case 1: return cast_e5m2_kernel<B, 1, 1, LPB>;
        case 2: return cast_e5m2_kernel<B, (MAXP >= 2 ? 2 : MAXP), 1, LPB>;
        case 3: return cast_e5m2_kernel<B, (MAXP >= 3 ? 3 : MAXP), 1, LPB>;
        default: return cast_e5m2_kernel<B, MAXP, 1, LPB>;
    }
}

template <int B, int LPB>
static fwd_fn pick_mxfp4_stat(int stat, int wpr, int npass)
{
    if (stat == STAT_MX) return pick_mxfp4<B, LPB, STAT_MX>(wpr, npass);
    if (stat == STAT_RMS) return pick_mxfp4<B, LPB, STAT_RMS>(wpr, npass);
    return pick_mxfp4<B, LPB, STAT_NONE>(wpr, npass);
}

template <int NPASS, int STAT>
static fwd_fn nvfp4_by_wpr(int wpr)
{
    switch (wpr) {
        case 1: return fwd_nvfp4_kernel<NPASS, 1, STAT>;
        case 2: return fwd_nvfp4_kernel<NPASS, 2, STAT>;
        case 3: return fwd_nvfp4_kernel<NPASS, 3, STAT>;
        case 4: return fwd_nvfp4_kernel<NPASS, 4, STAT>;
        case 5: return fwd_nvfp4_kernel<NPASS, 5, STAT>;
        case 6: return fwd_nvfp4_kernel<NPASS, 6, STAT>;
        case 7: return fwd_nvfp4_kernel<NPASS, 7, STAT>;
        case 8: return fwd_nvfp4_kernel<NPASS, 8, STAT>;
        case 16: return fwd_nvfp4_kernel<NPASS, 16, STAT>;
        default: return nullptr;
    }
}
template <int STAT>
static fwd_fn pick_nvfp4(int wpr, int npass)
{
    constexpr int MAXP = MXN_FWD_MAX_ELEMS / 16;
    if (npass == MAXP) return nvfp4_by_wpr<MAXP, STAT>(wpr);
    if (npass == MAXP / 2) return nvfp4_by_wpr<(MAXP >= 2 ? MAXP / 2 : 1), STAT>(wpr);
    if (npass == 1) return nvfp4_by_wpr<1, STAT>(wpr);
    return nullptr;
}

// Splits the K per-lane pieces of a row (B elements each) over WPR warps x NPASS passes (at most MXN_FWD_MAX_ELEMS
// elements per lane), choosing among the instantiated kernels by the fraction of idle lanes, with a handicap for
// splits that leave a lane little work when a row spans several warps (more warps, hence more synchronisation,
// per row).  Measured at 16384 rows: D = 7168, B = 32: 4 warps x 2 passes at 87.5 % beat 7 warps x 1 pass at 100 %;
// D = 2560, B = 16: 5 warps x 1 pass (16 elements per lane) at 100 % lost to 2 warps x 4 passes at 62.5 %.
static bool plan_row(int K, int B, bool fine, bool nvfp4, int* wpr, int* npass)
{
    const int maxp = MXN_FWD_MAX_ELEMS / B;
    int best_w = 0, best_p = 0;
    double best_cost = -1.0;
    const int* wl = fine ? kFineWpr : kCoarseWpr;
    const int nw = fine ? (int)(sizeof(kFineWpr) / sizeof(int)) : (int)(sizeof(kCoarseWpr) / sizeof(int));
    for (int wi = 0; wi < nw; ++wi) {
        const int w = wl[wi];
        for (int p = maxp; p >= 1; --p) {
            const bool reduced = p == 1 || (maxp >= 4 && p == maxp / 2);
            const bool exists = p == maxp || (nvfp4 ? reduced : (w == 1 || (fine && reduced)));
            const long lanes = (long)32 * w * p;
            if (!exists || lanes < K) continue;
            const int elems = p * B;   // per lane
            const double handicap = w == 1 || elems >= MXN_FWD_MAX_ELEMS ? 0.0 : elems >= MXN_FWD_MAX_ELEMS / 2 ? 0.15 : 0.45;
            const double cost = (double)(lanes - K) / (double)lanes + handicap;
            if (best_cost < 0.0 || cost < best_cost - 1e-9) {
                best_cost = cost;
                best_w = w;
                best_p = p;
            }
        }
    }
    if (best_cost < 0.0) return false;
    *wpr = best_w;
    *npass = best_p;
    return true;
}

bool fwd_shape_supported(int64_t D, int B)
{
    if (!(B == 16 || B == 32 || B == 64) || D <= 0 || D % B != 0 || D / B > (1 << 20)) return false;
    int wpr, npass;
    const int E = B == 64 ? 32 : B;
    return plan_row((int)(D / E), E, false, false, &wpr, &npass);   // the coarse set is the narrowest
}

cudaError_t launch_fwd(FwdParams P, int B, int stat, bool nvfp4, cudaStream_t stream)
{
    const bool mxfp4 = P.elem == ELEM_E2M1 && !nvfp4;
    const bool e5m2 = P.elem == ELEM_E5M2;
    const bool add = P.residual != nullptr;
    const int E = B == 64 ? 32 : B;   // elements per lane and pass; a block of 64 is shared by two lanes
    const bool fine = nvfp4 || (!mxfp4 && !e5m2 && !add && stat != STAT_POSTROUND && P.gain == nullptr &&
                                P.round == MXN_ROUND_RCEIL_POW2);
    P.pr_table = B == 16 ? 0 : B == 32 ? 1 : 2;
    P.chunks = P.K * (B / E);
    if (!plan_row(P.chunks, E, fine, nvfp4, &P.wpr, &P.npass)) return cudaErrorInvalidValue;
    P.tiles_per_row = (P.K + 3) / 4;
    {
        const int count = stat == STAT_RMS ? P.D : P.K;   // divisor of the row statistic
        P.inv_count = (count & (count - 1)) == 0 ? 1.0 / (double)count : 0.0;
    }
    const int warps = cta_warps(P.wpr);
    P.rows_per_cta = rows_per_cta(P.wpr);
    const bool has_gain = P.gain != nullptr;
    fwd_fn fn = nullptr;
    if (nvfp4) fn = stat == STAT_RMS ? pick_nvfp4<STAT_RMS>(P.wpr, P.npass) : pick_nvfp4<STAT_MX>(P.wpr, P.npass);
    else if (add) fn = B == 16 ? pick_add_mx<16, 1>(P.wpr, P.npass) : B == 32 ? pick_add_mx<32, 1>(P.wpr, P.npass) : pick_add_mx<32, 2>(P.wpr, P.npass);
    else if (e5m2) fn = B == 16 ? pick_e5m2<16, 1>(P.wpr, P.npass) : B == 32 ? pick_e5m2<32, 1>(P.wpr, P.npass) : pick_e5m2<32, 2>(P.wpr, P.npass);
    else if (mxfp4) fn = B == 16 ? pick_mxfp4_stat<16, 1>(stat, P.wpr, P.npass)
                       : B == 32 ? pick_mxfp4_stat<32, 1>(stat, P.wpr, P.npass) : pick_mxfp4_stat<32, 2>(stat, P.wpr, P.npass);
    else if (B == 16) fn = pick_round<16, 1>(P.round, stat, has_gain, P.wpr, P.npass);
    else if (B == 32) fn = pick_round<32, 1>(P.round, stat, has_gain, P.wpr, P.npass);
    else fn = pick_round<32, 2>(P.round, stat, has_gain, P.wpr, P.npass);
    if (fn == nullptr) return cudaErrorInvalidValue;
    const int64_t ctas = (P.T + P.rows_per_cta - 1) / P.rows_per_cta;
    if (ctas > 0x7FFFFFFF) return cudaErrorInvalidValue;
    // Programmatic stream serialisation: the kernel may be scheduled while the previous kernel of the
    // stream drains; it does not touch memory before that kernel has completed (pdl_prologue).
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(warps * kWarp);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fn, P);
}

// ---- host side of the post-round estimator: f, its inverse and the table --------------------------
// f(sigma) = E[max_i 2^floor(log2 |X_i|)] for B i.i.d. N(0, sigma^2) values
//          = sum_j 2^j (P(2^(j+1)) - P(2^j)),  P(t) = erf(t / (sigma sqrt 2))^B.
static double pr_expected_rounded_max(double sigma, int B)
{
    const double inv = 1.0 / (sigma * std::sqrt(2.0));
    const int centre = (int)std::floor(std::log2(sigma));
    double total = 0.0, below = std::pow(std::erf(std::ldexp(1.0, centre - 64) * inv), B);
    for (int j = centre - 64; j <= centre + 6; ++j) {
        const double above = std::pow(std::erf(std::ldexp(1.0, j + 1) * inv), B);
        total += std::ldexp(1.0, j) * (above - below);
        below = above;
    }
    return total;
}
static double pr_invert(double x, int B)
{
    double a = x / 8.0, b = x * 4.0;   // f(sigma) lies between sigma/2 and 4 sigma for these block sizes
    for (int it = 0; it < 200; ++it) {
        const double mid = 0.5 * (a + b);
        (pr_expected_rounded_max(mid, B) < x ? a : b) = mid;
    }
    return 0.5 * (a + b);
}

cudaError_t postround_prepare(int B)
{
    static std::mutex mtx;
    static bool done[64][3] = {};
    const int table = B == 16 ? 0 : B == 32 ? 1 : 2;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mtx);
    if (done[dev][table]) return cudaSuccess;
    double nodes[kPrIntervals + 1], values[kPrIntervals + 1], slopes[kPrIntervals];
    for (int i = 0; i <= kPrIntervals; ++i) {
        nodes[i] = i == kPrIntervals ? 2.0 : std::exp2((double)i / kPrIntervals);
        values[i] = pr_invert(nodes[i], B);
    }
    for (int i = 0; i < kPrIntervals; ++i) slopes[i] = (values[i + 1] - values[i]) / (nodes[i + 1] - nodes[i]);
    e = cudaMemcpyToSymbol(c_pr_nodes, nodes, sizeof nodes);
    if (e == cudaSuccess) e = cudaMemcpyToSymbol(c_pr_values, values, sizeof values, sizeof(double) * (kPrIntervals + 1) * table);
    if (e == cudaSuccess) e = cudaMemcpyToSymbol(c_pr_slopes, slopes, sizeof slopes, sizeof(double) * kPrIntervals * table);
    if (e == cudaSuccess) done[dev][table] = true;
    return e;
}

// ---- self test of the division shortcuts ------------------------------------------------------------
__global__ void selftest_division_kernel(unsigned long long* mismatches)
{
    const float divisors[10] = {6.0f, 448.0f, 1.0f, 1.125f, 1.25f, 1.375f, 1.5f, 1.625f, 1.75f, 1.875f};
    const uint64_t n = (uint64_t)200 << 23;   // exponent fields 27..226, every significand
    unsigned long long bad = 0;
    for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
        const float a = __uint_as_float((27u << 23) + (uint32_t)i);
        if (__float_as_uint(div_by_6(a)) != __float_as_uint(__fdiv_rn(a, 6.0f))) ++bad;
        const float c448 = 0x1.24924ap-9f;
        if (__float_as_uint(div_by_known(a, 448.0f, c448)) != __float_as_uint(__fdiv_rn(a, 448.0f))) ++bad;
#pragma unroll
        for (int m = 0; m < 8; ++m) {
            // E4M3 codes with exponent fields 1, 7 and 15 and significand m
            const uint32_t codes[3] = {(1u << 3) | m, (7u << 3) | m, (15u << 3) | (m == 7 ? 6u : m)};
#pragma unroll
            for (int j = 0; j < 3; ++j) {
                const float d = e4m3_to_f32(codes[j]);
                if (__float_as_uint(div_by_e4m3_normal(a, codes[j], d)) != __float_as_uint(__fdiv_rn(a, d))) ++bad;
            }
        }
        (void)divisors;
    }
    if (bad) atomicAdd(mismatches, bad);
}

cudaError_t selftest_division(unsigned long long* mismatches_host)
{
    unsigned long long* dev = nullptr;
    cudaError_t e = cudaMalloc(&dev, sizeof(unsigned long long));
    if (e != cudaSuccess) return e;
    e = cudaMemset(dev, 0, sizeof(unsigned long long));
    if (e == cudaSuccess) {
        selftest_division_kernel<<<148 * 8, 256>>>(dev);
        e = cudaDeviceSynchronize();
    }
    if (e == cudaSuccess) e = cudaMemcpy(mismatches_host, dev, sizeof(unsigned long long), cudaMemcpyDeviceToHost);
    cudaFree(dev);
    return e;
}

// number of bounded device-side waits that ran out since the library was loaded (synchronises);
// no kernel of this build waits on anything, so the counter stays 0
__device__ unsigned int g_timeouts = 0;
cudaError_t read_timeouts(unsigned int* out)
{
    return cudaMemcpyFromSymbol(out, g_timeouts, sizeof(unsigned int));
}

}  // namespace mxn
