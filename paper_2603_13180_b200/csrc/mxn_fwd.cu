// Forward kernels: MXCast, fused RMSNorm+MXCast (Algorithm 1) and MXNorm (Algorithm 2) with
// E4M3 codes / E8M0 scales, and the NVFP4 variant of MXNorm (E2M1 codes / E4M3 scales).
//
// Work decomposition (memory-bound streaming map with one scalar reduction per row):
//   * a row is handled by a "row group" of WPR warps (1 for D <= 4096 at B = 32) and stays in
//     registers between the statistics phase and the quantise phase - every input byte is read
//     from HBM exactly once, with 32-byte loads that bypass L1;
//   * one lane owns one whole block per pass (B contiguous elements = 2B bytes), so the block
//     absmax needs no cross-lane traffic, the scale is computed once per block, a warp writes
//     32 consecutive scale bytes and 32*B consecutive code bytes per pass;
//   * the only cross-lane step is the row statistic: K = D/B block values (MXNorm) instead of
//     D squares (RMSNorm), reduced in binary64 by shuffles (and through shared memory when a row
//     spans several warps).
#include "mxn_device.cuh"
#include "mxn_internal.h"

namespace mxn {

constexpr int kThreads = 128;   // 4 warps per CTA; rows per CTA = 4 / WPR (WPR = 8 uses 256 threads)

// row statistic -> (r, rho) ; one value per row group ------------------------------------------
template <int STAT>
__device__ __forceinline__ void finish_stat(double s, const FwdParams& P, float& r, float& rho)
{
    if (STAT == STAT_MX) {
        // G = (1/K sum m^p)^(1/p); r~ = fl32(coef * G); rho~ = 1 / fl32(r~ + eps)
        double mean = __ddiv_rn(s, (double)P.K);
        double G = P.p == 2 ? __dsqrt_rn(mean) : mean;
        r = __double2float_rn(__dmul_rn((double)P.coef, G));
        float den = __fadd_rn(r, P.eps);
        rho = den == 0.0f ? 0.0f : __fdiv_rn(1.0f, den);
    } else if (STAT == STAT_RMS) {
        // r = fl32(sqrt(mean x^2 + eps)); rho = 1 / r
        double ms = __ddiv_rn(s, (double)P.D);
        r = __double2float_rn(__dsqrt_rn(__dadd_rn(ms, (double)P.eps)));
        rho = r == 0.0f ? 0.0f : __fdiv_rn(1.0f, r);
    } else {
        r = 1.0f;
        rho = 1.0f;
    }
}

// sum of one double per warp over the WPR warps of a row group, in a fixed order
__device__ __forceinline__ double group_sum(double v, int wpr, int group, int w, double* smem)
{
    v = warp_sum(v);
    if (wpr > 1) {
        if ((threadIdx.x & 31) == 0) smem[group * 8 + w] = v;
        group_barrier(1 + group, wpr * kWarp);
        double t = smem[group * 8];
        for (int i = 1; i < wpr; ++i) t = __dadd_rn(t, smem[group * 8 + i]);
        v = t;
    }
    return v;
}

template <int B, int NPASS, int STAT, bool GAIN>
__global__ void __launch_bounds__(256) fwd_e4m3_kernel(const FwdParams P)
{
    constexpr int W = B / 2;   // 32-bit words (bf16 pairs) per block
    __shared__ double red[8 * 8];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int wpr = P.wpr;
    const int group = warp / wpr, w = warp - group * wpr;
    const int64_t row = (int64_t)blockIdx.x * P.rows_per_cta + group;
    if (row >= P.T) return;   // whole row group leaves together

    const uint16_t* xrow = P.x + row * P.D;
    uint32_t xr[NPASS][W];
    float m[NPASS];

    // ---- load the row slice: block k = (pass*WPR + w)*32 + lane -------------------------------
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        const int k = (i * wpr + w) * kWarp + lane;
        if (k < P.K) {
            const uint16_t* p = xrow + (int64_t)k * B;
#pragma unroll
            for (int v = 0; v < W / 8; ++v) ld_v8(p + v * 16, &xr[i][v * 8]);
        } else {
#pragma unroll
            for (int j = 0; j < W; ++j) xr[i][j] = 0u;
        }
    }

    // ---- phase 1: block absmaxes and the row statistic ---------------------------------------
    double stat = 0.0;
    float ss0 = 0.f, ss1 = 0.f, ss2 = 0.f, ss3 = 0.f;
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        uint32_t m2 = absmax_bf16x2(xr[i][0], xr[i][1]);
#pragma unroll
        for (int j = 2; j < W; ++j) m2 = absmax_bf16x2(m2, xr[i][j]);
        m[i] = hmax_abs_to_f32(m2);
        if (STAT == STAT_MX) {
            double md = (double)m[i];
            stat = P.p == 2 ? __fma_rn(md, md, stat) : __dadd_rn(stat, md);   // m^2 is exact in binary64
        }
        if (STAT == STAT_RMS) {
#pragma unroll
            for (int j = 0; j < W; j += 2) {
                float a = bf16_lo(xr[i][j]), b = bf16_hi(xr[i][j]);
                float c = bf16_lo(xr[i][j + 1]), d = bf16_hi(xr[i][j + 1]);
                ss0 = __fmaf_rn(a, a, ss0);
                ss1 = __fmaf_rn(b, b, ss1);
                ss2 = __fmaf_rn(c, c, ss2);
                ss3 = __fmaf_rn(d, d, ss3);
            }
        }
    }
    float r = 1.0f, rho = 1.0f;
    if (STAT != STAT_NONE) {
        if (STAT == STAT_RMS) stat = (double)ss0 + (double)ss1 + ((double)ss2 + (double)ss3);
        stat = group_sum(stat, wpr, group, w, red);
        finish_stat<STAT>(stat, P, r, rho);
        if (P.rms_out != nullptr && w == 0 && lane == 0) P.rms_out[row] = r;
    }
    const bool rho_normal = is_normal_f32(rho);

    // ---- phase 2: scales and codes -----------------------------------------------------------
    uint8_t* crow = P.codes + row * P.D;
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        const int k = (i * wpr + w) * kWarp + lane;
        const bool active = k < P.K;
        uint32_t out[W / 2];
        uint32_t sb;
        if (!GAIN) {
            // a = fl32(m * rho) is also the absmax of fl32(x * rho): rounding is monotone
            const float a = __fmul_rn(m[i], rho);
            sb = e8m0_scale(a, P.round);
            const float inv = inv_scale(sb);
            // q = fl32(x*rho) * 2^(127-sb).  When neither factor product leaves the normal range the
            // two roundings collapse into the single product x * (rho * 2^(127-sb)).
            const float f = __fmul_rn(rho, inv);
            const bool fast = sb >= 16u && rho_normal && is_normal_f32(f);
            if (__all_sync(0xFFFFFFFFu, fast || !active)) {
#pragma unroll
                for (int j = 0; j < W; j += 2)
                    out[j / 2] = cvt_e4m3x4(__fmul_rn(bf16_lo(xr[i][j]), f), __fmul_rn(bf16_hi(xr[i][j]), f),
                                            __fmul_rn(bf16_lo(xr[i][j + 1]), f), __fmul_rn(bf16_hi(xr[i][j + 1]), f));
            } else {
#pragma unroll
                for (int j = 0; j < W; j += 2)
                    out[j / 2] = cvt_e4m3x4(__fmul_rn(__fmul_rn(bf16_lo(xr[i][j]), rho), inv),
                                            __fmul_rn(__fmul_rn(bf16_hi(xr[i][j]), rho), inv),
                                            __fmul_rn(__fmul_rn(bf16_lo(xr[i][j + 1]), rho), inv),
                                            __fmul_rn(__fmul_rn(bf16_hi(xr[i][j + 1]), rho), inv));
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
            sb = e8m0_scale(my, P.round);
            const float inv = inv_scale(sb);
#pragma unroll
            for (int j = 0; j < W; j += 2) {
                const float y0 = __fmul_rn(__fmul_rn(bf16_lo(xr[i][j]), rho), bf16_lo(gr[j]));
                const float y1 = __fmul_rn(__fmul_rn(bf16_hi(xr[i][j]), rho), bf16_hi(gr[j]));
                const float y2 = __fmul_rn(__fmul_rn(bf16_lo(xr[i][j + 1]), rho), bf16_lo(gr[j + 1]));
                const float y3 = __fmul_rn(__fmul_rn(bf16_hi(xr[i][j + 1]), rho), bf16_hi(gr[j + 1]));
                out[j / 2] = cvt_e4m3x4(__fmul_rn(y0, inv), __fmul_rn(y1, inv), __fmul_rn(y2, inv), __fmul_rn(y3, inv));
            }
        }
        if (active) {
            uint8_t* cp = crow + (int64_t)k * B;
            if (B == 16) {
                st_v4(cp, out);
            } else {
#pragma unroll
                for (int v = 0; v < W / 16; ++v) st_v8(cp + v * 32, &out[v * 8]);
            }
            P.scales[scale_offset(row, k, P.K, P.tiles_per_row, P.layout)] = (uint8_t)sb;
        }
    }
}

// NVFP4: B = 16 (one 32-byte load per block), E4M3 block scales, E2M1 codes two per byte.
template <int NPASS>
__global__ void __launch_bounds__(256) fwd_nvfp4_kernel(const FwdParams P)
{
    constexpr int B = 16, W = 8;
    __shared__ double red[8 * 8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int wpr = P.wpr;
    const int group = warp / wpr, w = warp - group * wpr;
    const int64_t row = (int64_t)blockIdx.x * P.rows_per_cta + group;
    if (row >= P.T) return;

    const uint16_t* xrow = P.x + row * P.D;
    uint32_t xr[NPASS][W];
    float m[NPASS];
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        const int k = (i * wpr + w) * kWarp + lane;
        if (k < P.K) {
            ld_v8(xrow + (int64_t)k * B, xr[i]);
        } else {
#pragma unroll
            for (int j = 0; j < W; ++j) xr[i][j] = 0u;
        }
    }
    double stat = 0.0;
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        uint32_t m2 = absmax_bf16x2(xr[i][0], xr[i][1]);
#pragma unroll
        for (int j = 2; j < W; ++j) m2 = absmax_bf16x2(m2, xr[i][j]);
        m[i] = hmax_abs_to_f32(m2);
        double md = (double)m[i];
        stat = P.p == 2 ? __fma_rn(md, md, stat) : __dadd_rn(stat, md);
    }
    stat = group_sum(stat, wpr, group, w, red);
    float r, rho;
    finish_stat<STAT_MX>(stat, P, r, rho);
    if (P.rms_out != nullptr && w == 0 && lane == 0) P.rms_out[row] = r;
    const float rho_g = __fmul_rn(rho, P.global_scale);

    uint8_t* crow = P.codes + row * (P.D / 2);
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        const int k = (i * wpr + w) * kWarp + lane;
        // block scale = E4M3(fl32(fl32(a/6) * global_scale)), a = fl32(m * rho~)
        const float a = __fmul_rn(m[i], rho);
        const float t = __fmul_rn(__fdiv_rn(a, 6.0f), P.global_scale);
        const uint32_t sc = cvt_e4m3x2(t, 0.0f) & 0xFFu;
        const float d = e4m3_to_f32(sc);
        const float inv = d == 0.0f ? 0.0f : __fdiv_rn(rho_g, d);
        uint32_t out[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t word = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t xw = xr[i][h * 4 + j];
                word |= cvt_e2m1x2(__fmul_rn(bf16_lo(xw), inv), __fmul_rn(bf16_hi(xw), inv)) << (8 * j);
            }
            out[h] = word;
        }
        if (k < P.K) {
            st_v2(crow + (int64_t)k * 8, out);
            P.scales[scale_offset(row, k, P.K, P.tiles_per_row, P.layout)] = (uint8_t)sc;
        }
    }
}

// ---- dispatch ---------------------------------------------------------------------------------
typedef void (*fwd_fn)(const FwdParams);

template <int B, int STAT, bool GAIN>
static fwd_fn pick_npass(int npass)
{
    constexpr int MAXP = 128 / B;
    switch (npass) {
        case 1: return fwd_e4m3_kernel<B, 1, STAT, GAIN>;
        case 2: return fwd_e4m3_kernel<B, 2, STAT, GAIN>;
        case 3: if (MAXP >= 3) return fwd_e4m3_kernel<B, (MAXP >= 3 ? 3 : 1), STAT, GAIN>; break;
        case 4: if (MAXP >= 4) return fwd_e4m3_kernel<B, (MAXP >= 4 ? 4 : 1), STAT, GAIN>; break;
        case 5: case 6: if (MAXP >= 6) return fwd_e4m3_kernel<B, (MAXP >= 6 ? 6 : 1), STAT, GAIN>; break;
        case 7: case 8: if (MAXP >= 8) return fwd_e4m3_kernel<B, (MAXP >= 8 ? 8 : 1), STAT, GAIN>; break;
        default: break;
    }
    return nullptr;
}
template <int B>
static fwd_fn pick_stat(int stat, bool gain, int npass)
{
    switch (stat) {
        case STAT_NONE: return pick_npass<B, STAT_NONE, false>(npass);
        case STAT_RMS: return gain ? pick_npass<B, STAT_RMS, true>(npass) : pick_npass<B, STAT_RMS, false>(npass);
        case STAT_MX: return gain ? pick_npass<B, STAT_MX, true>(npass) : pick_npass<B, STAT_MX, false>(npass);
        default: return nullptr;
    }
}

// Splits K blocks per row over WPR warps x NPASS passes with at most 128 elements per lane.
static bool plan_row(int K, int B, int* wpr, int* npass)
{
    const int maxp = 128 / B;
    int w = 1;
    while ((K + 32 * w - 1) / (32 * w) > maxp) {
        w *= 2;
        if (w > 8) return false;
    }
    *wpr = w;
    *npass = (K + 32 * w - 1) / (32 * w);
    return true;
}

bool fwd_shape_supported(int64_t D, int B)
{
    if (!(B == 16 || B == 32 || B == 64) || D <= 0 || D % B != 0 || D / B > (1 << 20)) return false;
    int wpr, npass;
    return plan_row((int)(D / B), B, &wpr, &npass);
}

cudaError_t launch_fwd(FwdParams P, int B, int stat, bool nvfp4, cudaStream_t stream)
{
    if (!plan_row(P.K, B, &P.wpr, &P.npass)) return cudaErrorInvalidValue;
    const int warps = P.wpr == 8 ? 8 : 4;
    P.rows_per_cta = warps / P.wpr;
    P.tiles_per_row = (P.K + 3) / 4;
    fwd_fn fn = nullptr;
    if (nvfp4) {
        switch (P.npass) {
            case 1: fn = fwd_nvfp4_kernel<1>; break;
            case 2: fn = fwd_nvfp4_kernel<2>; break;
            case 3: fn = fwd_nvfp4_kernel<3>; break;
            case 4: fn = fwd_nvfp4_kernel<4>; break;
            case 5: case 6: fn = fwd_nvfp4_kernel<6>; break;
            default: fn = fwd_nvfp4_kernel<8>; break;
        }
    } else if (B == 16) {
        fn = pick_stat<16>(stat, P.gain != nullptr, P.npass);
    } else if (B == 32) {
        fn = pick_stat<32>(stat, P.gain != nullptr, P.npass);
    } else {
        fn = pick_stat<64>(stat, P.gain != nullptr, P.npass);
    }
    if (fn == nullptr) return cudaErrorInvalidValue;
    const int64_t ctas = (P.T + P.rows_per_cta - 1) / P.rows_per_cta;
    if (ctas > 0x7FFFFFFF) return cudaErrorInvalidValue;
    fn<<<(unsigned)ctas, warps * kWarp, 0, stream>>>(P);
    return cudaGetLastError();
}

}  // namespace mxn
