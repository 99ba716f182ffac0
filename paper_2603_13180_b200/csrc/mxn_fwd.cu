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
//     faster on B200 than resident CTAs, with or without TMA staging;
//   * the CTAs of the first wave ask for their rows in L2 (a bulk prefetch hint) before they wait for the
//     previous kernel of the stream, so that the DRAM idling during that kernel's tail already fetches
//     this kernel's first rows; no value is read before the wait.
#include <cmath>
#include <mutex>

#include "mxn_device.cuh"
#include "mxn_internal.h"
#include "mxn_row.cuh"
#include "mxn_fwd_common.cuh"

namespace mxn {

template <int B, int NPASS, int WPR, int STAT, bool GAIN, bool PAPER, int LPB = 1>
__global__ void __launch_bounds__(cta_warps(WPR) * 32, fwd_min_ctas(WPR)) fwd_e4m3_kernel(const FwdParams P)
{
    __shared__ double red[WPR > 1 ? cta_warps(WPR) : 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int group = warp / WPR, w = warp - group * WPR;
    const int64_t row = (int64_t)blockIdx.x * rows_per_cta(WPR) + group;
    prefetch_row(P.x, row, P, w, lane);
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
    prefetch_row(P.x, row, P, w, lane);
    prefetch_row(P.residual, row, P, w, lane);
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
__global__ void __launch_bounds__(cta_warps(WPR) * 32, fwd_min_ctas(WPR)) cast_e5m2_kernel(const FwdParams P)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int group = warp / WPR, w = warp - group * WPR;
    const int64_t row = (int64_t)blockIdx.x * rows_per_cta(WPR) + group;
    prefetch_row(P.x, row, P, w, lane);
    pdl_prologue();
    if (row >= P.T) return;
    uint32_t xr[NPASS][B / 2];
    float m[NPASS];
    load_row_direct<B, NPASS>(xr, P.x + row * P.D, P.chunks, WPR, w, lane);
    (void)block_stats<B, NPASS, STAT_NONE, LPB>(xr, m, 2, lane);
    quantise_store_e4m3<B, NPASS, WPR, false, true, 2, LPB>(xr, m, 1.0f, P, row, w, lane);
}

// ---- one warp per run of RPW short rows ------------------------------------------------------------------------------
// One warp, no shared memory.  The warp takes RPW consecutive rows of CH pieces each (E = 16 elements per piece, LPB lanes
// per block) as one contiguous run of RPW * CH pieces: piece j of the run goes to pass j / 32, lane j % 32, so every lane
// of every pass is busy when RPW * CH = 32 NPASS, however the rows fall on the passes (CH is a compile-time constant:
// the row of a piece is a constant division).  Used for rows that no warps-per-row split fills (D = 2560: CH = 160, one
// row per warp; D = 1280: CH = 80, two rows per warp; D = 1536: three passes) and for rows too short to keep a warp's
// loads in flight (D = 512: four rows per warp; D = 768: two); see one_warp_shape.  The row statistics are independent
// shuffle reductions, one per row.
template <int E, int LPB, int NPASS, int RPW, int CH, int STAT, int FMT>
__global__ void __launch_bounds__(MXN_FWD_WARPS * 32, 32 / MXN_FWD_WARPS) fwd_multi_kernel(const FwdParams P)
{
    constexpr int W = E / 2;
    static_assert(RPW * CH <= 32 * NPASS && CH % LPB == 0 && (E == 16 || E == 32), "the run fits the warp's passes; 32- or 64-byte pieces");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row0 = ((int64_t)blockIdx.x * MXN_FWD_WARPS + warp) * RPW;
    const int nrows = (int)(P.T - row0 < RPW ? P.T - row0 : RPW);     // <= 0 past the end
    if (lane == 0 && blockIdx.x < kFirstWaveCtas && nrows > 0) prefetch_l2_bulk(P.x + row0 * P.D, (uint32_t)(nrows * CH) * (E * 2u));
    pdl_prologue();
    if (nrows <= 0) return;
    const int npieces = nrows * CH;
    const int64_t first = row0 * CH;

    uint32_t xr[NPASS][W];
    float m[NPASS];
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        const int j = i * 32 + lane;
        if (j < npieces) {
            const uint16_t* p = P.x + (first + j) * E;
#pragma unroll
            for (int v = 0; v < W / 8; ++v) ld_v8(p + v * 16, &xr[i][v * 8]);
        } else {
#pragma unroll
            for (int q = 0; q < W; ++q) xr[i][q] = 0u;
        }
    }
    double stat[RPW];
    float2 ssa[RPW], ssb[RPW];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
        stat[r] = 0.0;
        ssa[r] = ssb[r] = make_float2(0.f, 0.f);
    }
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        const int rl = (i * 32 + lane) / CH;
        uint32_t m2 = absmax_bf16x2(xr[i][0], xr[i][1]);
#pragma unroll
        for (int q = 2; q < W; ++q) m2 = absmax_bf16x2(m2, xr[i][q]);
        m[i] = hmax_abs_to_f32(m2);
#pragma unroll
        for (int o = 1; o < LPB; o <<= 1) m[i] = fmaxf(m[i], __shfl_xor_sync(0xFFFFFFFFu, m[i], o));
        const float mc = (LPB == 1 || (lane & (LPB - 1)) == 0) ? m[i] : 0.0f;
        float2 sa = make_float2(0.f, 0.f), sb2 = make_float2(0.f, 0.f);
        if (STAT == STAT_RMS) {
#pragma unroll
            for (int q = 0; q < W; q += 2) {
                const float2 a = bf16x2_to_f32x2(xr[i][q]), b = bf16x2_to_f32x2(xr[i][q + 1]);
                sa = __ffma2_rn(a, a, sa);
                sb2 = __ffma2_rn(b, b, sb2);
            }
        }
#pragma unroll
        for (int r = 0; r < RPW; ++r) {
            if (i * 32 / CH > r || (i * 32 + 31) / CH < r) continue;       // this pass holds no piece of row r (compile time)
            const bool mine = RPW == 1 || rl == r;
            if (STAT == STAT_MX) {
                const double md = mine ? (double)mc : 0.0;                    // adding 0 is exact
                stat[r] = P.p == 2 ? __fma_rn(md, md, stat[r]) : __dadd_rn(stat[r], md);
            }
            if (STAT == STAT_RMS) {
                ssa[r] = __fadd2_rn(ssa[r], mine ? sa : make_float2(0.f, 0.f));
                ssb[r] = __fadd2_rn(ssb[r], mine ? sb2 : make_float2(0.f, 0.f));
            }
        }
    }
    if (STAT == STAT_RMS) forget_unpacked<NPASS, W>(xr);
    float rho[RPW];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
        rho[r] = 1.0f;
        if (STAT != STAT_NONE) {
            if (STAT == STAT_RMS) stat[r] = (double)ssa[r].x + (double)ssa[r].y + ((double)ssb[r].x + (double)ssb[r].y);
            float rr;
            finish_stat<STAT>(warp_sum(stat[r]), P, rr, rho[r]);
            if (P.rms_out != nullptr && lane == 0 && r < nrows) P.rms_out[row0 + r] = rr;
        }
    }
    const float rcp_sig = FMT == 2 ? kRcpE4M3Significand[lane & 7] : 0.0f;
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        const int j = i * 32 + lane;
        const bool active = j < npieces;
        const int rl = j / CH;
        float rh = rho[0];
#pragma unroll
        for (int r = 1; r < RPW; ++r) rh = rl == r ? rho[r] : rh;
        uint32_t sbyte;
        if constexpr (FMT == 0) {
            uint32_t out[W / 2];
            sbyte = quantise_piece_fp8<E, true, 0>(xr[i], m[i], rh, is_normal_f32(rh), active, 0, out);
            if (active) {
                uint8_t* cp = P.codes + (first + j) * E;
                if constexpr (E == 16) st_v4(cp, out);
                else st_v8(cp, out);
            }
        } else if constexpr (FMT == 1) {
            uint32_t out[W / 4];
            sbyte = quantise_piece_mxfp4<E>(xr[i], m[i], rh, is_normal_f32(rh), active, out);
            if (active) {
                uint8_t* cp = P.codes + (first + j) * (E / 2);
                if constexpr (E == 16) st_v2(cp, out);
                else st_v4(cp, out);
            }
        } else {
            uint32_t out[2];
            const float rho_g = __fmul_rn(rh, P.global_scale);
            sbyte = quantise_piece_nvfp4(xr[i], m[i], rh, rho_g, in_division_window(rho_g), rcp_sig, P.global_scale, active, out);
            if (active) st_v2(P.codes + (first + j) * 8, out);
        }
        if (active && (LPB == 1 || (lane & (LPB - 1)) == 0)) {
            int64_t off;
            if (P.layout == MXN_SCALES_ROWMAJOR) {
                off = (first + j) / LPB;                       // scales of consecutive rows are contiguous too
            } else {
                const int64_t row = row0 + rl;
                const int kb = (j - rl * CH) / LPB, rr = (int)(row & 127);
                off = ((row >> 7) * P.tiles_per_row + (kb >> 2)) * 512 + (rr & 31) * 16 + (rr >> 5) * 4 + (kb & 3);
            }
            P.scales[off] = (uint8_t)sbyte;
        }
    }
}

// ---- dispatch ---------------------------------------------------------------------------------

// In the templates below B is the number of elements a lane holds per pass and LPB the lanes per block
// (block size of the format = B * LPB: 16 = 16x1, 32 = 32x1, 64 = 32x2).
// The E4M3 kernels (every rounding rule, with and without gain), MXFP4 and NVFP4 exist for every number of
// warps per row in kFineWpr, so that hidden sizes of the form {3,5,7} * 2^r fill their lanes; the
// other variants (post-round statistic, residual add, E5M2) exist for power-of-two warps per row only.
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
    constexpr bool FINE = STAT != STAT_POSTROUND;
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
static fwd_fn pick_stat(int stat, int wpr, int npass)
{
    switch (stat) {
        case STAT_NONE: return pick_e4m3<B, LPB, STAT_NONE, false, PAPER>(wpr, npass);
        case STAT_RMS: return pick_e4m3<B, LPB, STAT_RMS, false, PAPER>(wpr, npass);
        case STAT_MX: return pick_e4m3<B, LPB, STAT_MX, false, PAPER>(wpr, npass);
        case STAT_POSTROUND: return !PAPER ? nullptr : pick_e4m3<B, LPB, STAT_POSTROUND, false, true>(wpr, npass);
        default: return nullptr;
    }
}
template <int B, int LPB>
static fwd_fn pick_round(int round, int stat, int wpr, int npass)
{
    return round == MXN_ROUND_RCEIL_POW2 ? pick_stat<B, LPB, true>(stat, wpr, npass) : pick_stat<B, LPB, false>(stat, wpr, npass);
}
// With a gain a lane always holds 16-element pieces (a block of 32 or 64 is shared by 2 or 4 lanes): the products
// x * rho * gamma of a piece stay in registers between the block maximum and the conversion, and 16 of them fit the
// 64 registers that 32 resident warps per SM allow, 32 do not (measured at [16384, 4096], block 32: 37.3 us as 32-element
// pieces, 32.2 us as 16-element pieces; 42.7 us before, with scalar arithmetic and no register limit).
template <int LPB, bool PAPER>
static fwd_fn pick_gain_stat(int stat, int wpr, int npass)
{
    switch (stat) {
        case STAT_RMS: return pick_e4m3<16, LPB, STAT_RMS, true, PAPER>(wpr, npass);
        case STAT_MX: return pick_e4m3<16, LPB, STAT_MX, true, PAPER>(wpr, npass);
        default: return nullptr;
    }
}
// (the rounding rule read at run time instead of compiled in costs the gain kernels 3-5 %, the others nothing measurable)
template <int LPB>
static fwd_fn pick_gain_round(int round, int stat, int wpr, int npass)
{
    return round == MXN_ROUND_RCEIL_POW2 ? pick_gain_stat<LPB, true>(stat, wpr, npass) : pick_gain_stat<LPB, false>(stat, wpr, npass);
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



// The one-warp kernel with 16-element pieces is used where it measured faster than the row-group kernels (all variants
// at 64 registers; [16384, D] and [65536, D]):
//   D = 2560 (160 pieces, one row per warp: five passes of one warp instead of three warps x one pass or two warps x four
//     passes): every format, 8-16 % faster;
//   D = 512 (four rows per warp; 32-element pieces for blocks of 32 and 64 with E8M0 scales, 3-16 % faster than
//     16-element pieces there): every format and statistic, 8-58 % faster at 65536 rows, -8 ... +18 % at 16384;
//   D = 256 (eight rows per warp, pieces as for D = 512): every format, 10-127 % faster from 32768 rows on (a row of
//     256 elements leaves three quarters of a warp's lanes idle in the row-group kernels);
//   D = 768 (48 pieces, two rows per warp): blocks of 16 only (1-19 % faster; blocks of 32 and 64 are level, also as
//     32-element pieces);
//   D = 1280 (80 pieces, two rows per warp): blocks of 16 with the MXNorm statistic (4-11 % faster; the sum of squares
//     loses 2-9 % there, blocks of 32 / 64 gain 4 % at 65536 rows and lose 4 % at 16384), and NVFP4 (level);
//   D = 1536 (96 pieces, one row per warp, three passes): NVFP4 only (6-9 % faster; the E8M0-scaled formats are level).
// Measured and not kept: two rows per warp at D = 1024 (16-element pieces: -9 ... +6 %; 32-element pieces: -5 ... +3 %), 8-element pieces with four lanes per
// block (D = 1280: 5.1 -> 3.8 TB/s, D = 1792: 6.1 -> 4.0), and CTA tiles of whole rows packed across warps through shared
// memory (two CTA-wide barriers per tile: slower than one row per row group at every size but D = 2560).
struct MultiShape { int rpw, ch, e; };   // rows per warp, pieces per row, elements per piece
static MultiShape one_warp_shape(int64_t T, int64_t D, int B, bool nvfp4, int stat)
{
    if (D == 2560) return {1, 160, 16};
    if (D == 1280 && nvfp4) return {2, 80, 16};
    if (D == 1536 && nvfp4) return {1, 96, 16};
    // several rows per warp mean as many times fewer CTAs: below about 12 thousand rows (24 thousand for eight rows per
    // warp) the grid no longer fills the SMs (D = 1280, blocks of 16: 9 % slower at 8192 rows, 6-17 % faster from 16384 on;
    // D = 256: -10 ... +27 % at 16384 rows, 10-127 % faster from 32768 on)
    if (T < 12288) return {0, 0, 0};
    if (D == 256 && T >= 24576) return B >= 32 && !nvfp4 ? MultiShape{8, 8, 32} : MultiShape{8, 16, 16};
    if (D == 512) return B >= 32 && !nvfp4 ? MultiShape{4, 16, 32} : MultiShape{4, 32, 16};
    if (D == 768 && B == 16) return {2, 48, 16};
    if (D == 1280 && B == 16 && stat == STAT_MX) return {2, 80, 16};
    return {0, 0, 0};
}

template <int LPB, int FMT, int STAT>
static fwd_fn multi_by_rows(int ch, int e)
{
    if constexpr (LPB >= 2 && FMT != 2) {   // 32-element pieces: a block of 32 is one lane's, a block of 64 two lanes'
        if (e == 32) return ch == 16 ? fwd_multi_kernel<32, LPB / 2, 2, 4, 16, STAT, FMT> : ch == 8 ? fwd_multi_kernel<32, LPB / 2, 2, 8, 8, STAT, FMT> : nullptr;
    }
    if (e != 16) return nullptr;
    if (ch == 160) return fwd_multi_kernel<16, LPB, 5, 1, 160, STAT, FMT>;
    if (ch == 32) return fwd_multi_kernel<16, LPB, 4, 4, 32, STAT, FMT>;
    if (ch == 16) return fwd_multi_kernel<16, LPB, 4, 8, 16, STAT, FMT>;
    if constexpr (LPB == 1) {
        if (ch == 48) return fwd_multi_kernel<16, LPB, 3, 2, 48, STAT, FMT>;
        if constexpr (FMT == 2 || STAT == STAT_MX) {
            if (ch == 80) return fwd_multi_kernel<16, LPB, 5, 2, 80, STAT, FMT>;
        }
        if constexpr (FMT == 2) {
            if (ch == 96) return fwd_multi_kernel<16, LPB, 3, 1, 96, STAT, FMT>;
        }
    }
    return nullptr;
}
template <int FMT, int STAT>
static fwd_fn pick_multi(int B, int ch, int e)
{
    if constexpr (FMT == 2) return multi_by_rows<1, 2, STAT>(ch, e);
    else return B == 16 ? multi_by_rows<1, FMT, STAT>(ch, e) : B == 32 ? multi_by_rows<2, FMT, STAT>(ch, e) : multi_by_rows<4, FMT, STAT>(ch, e);
}
template <int FMT>
static fwd_fn pick_multi_stat(int B, int stat, int ch, int e)
{
    return stat == STAT_MX ? pick_multi<FMT, STAT_MX>(B, ch, e) : stat == STAT_RMS ? pick_multi<FMT, STAT_RMS>(B, ch, e) : pick_multi<FMT, STAT_NONE>(B, ch, e);
}


// Splits the K per-lane pieces of a row (B elements each) over WPR warps x NPASS passes (at most MXN_FWD_MAX_ELEMS
// elements per lane), choosing among the instantiated kernels by the fraction of idle lanes, with a handicap for
// splits that leave a lane little work when a row spans several warps (more warps, hence more synchronisation,
// per row).  Measured at 16384 rows: D = 7168, B = 32: 4 warps x 2 passes at 87.5 % beat 7 warps x 1 pass at 100 %;
// D = 2560, B = 16: 5 warps x 1 pass (16 elements per lane) at 100 % lost to 2 warps x 4 passes at 62.5 %.
// Measured at 32768 rows, every format: D = 5120: 3 warps x the full 64 elements at 83 % beat 5 warps x 32 elements at
// 100 % by 3-6 %; D = 3072 with 32-element pieces: 2 warps x 64 at 75 % beat 3 warps x 32 at 100 % by 2 %, with
// 16-element pieces the two are level; D = 2560 with 16-element pieces and a gain: 2 warps x 64 at 62.5 % beat 3 warps x 32
// at 83 % (26.3 against 28.2 us at 16384 rows).  Hence the handicap of a half-filled lane: 0.26 and 0.22.
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
            const double handicap = w == 1 || elems >= MXN_FWD_MAX_ELEMS ? 0.0 : elems >= MXN_FWD_MAX_ELEMS / 2 ? (B == 32 ? 0.26 : 0.22) : 0.45;
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

// Everything a launch needs that does not depend on the pointers: the row plan written into P, the kernel, the grid and
// the CTA size.  Kept apart from the launch so that the host-side self-test can walk every supported shape.
static bool select_fwd(FwdParams& P, int B, int stat, bool nvfp4, fwd_fn* fn_out, int64_t* ctas_out, int* threads_out)
{
    const bool mxfp4 = P.elem == ELEM_E2M1 && !nvfp4;
    const bool e5m2 = P.elem == ELEM_E5M2;
    const bool add = P.residual != nullptr;
#ifdef MXN_NVFP4_NO_PAIR
    const bool nv_pair = false;
#else
    // NVFP4 rows of an even number of blocks: a lane owns two adjacent blocks (about a fifth fewer instructions).  Measured
    // 0-2 % faster than one block per lane up to D = 12288, level at 14336 and 1 % slower at 16384, hence the limit.
    const bool nv_pair = nvfp4 && P.K % 2 == 0 && P.D < 12288;
#endif
    const bool has_gain = P.gain != nullptr && P.elem == ELEM_E4M3 && !add;
    // elements per lane and pass; a block of 64 is shared by two lanes, with a gain every block by lanes of 16 elements
    const int E = nv_pair ? 32 : has_gain ? 16 : B == 64 ? 32 : B;
    const bool fine = nvfp4 || mxfp4 || (!e5m2 && !add && stat != STAT_POSTROUND);
    P.pr_table = B == 16 ? 0 : B == 32 ? 1 : 2;
    P.chunks = nv_pair ? P.K / 2 : P.K * (B / E);
    if (!plan_row(P.chunks, E, fine, nvfp4 && !nv_pair, &P.wpr, &P.npass)) return false;
    P.tiles_per_row = (P.K + 3) / 4;
    {
        const int count = stat == STAT_RMS ? P.D : P.K;   // divisor of the row statistic
        P.inv_count = (count & (count - 1)) == 0 ? 1.0 / (double)count : 0.0;
    }
    const int warps = cta_warps(P.wpr);
    P.rows_per_cta = rows_per_cta(P.wpr);
    fwd_fn fn = nullptr;
    // (the one-warp kernel has the paper's rounding rule compiled in and takes no gain)
    if (const MultiShape ms = one_warp_shape(P.T, P.D, B, nvfp4, stat); ms.rpw > 0 && !has_gain && (nvfp4 || mxfp4 || P.round == MXN_ROUND_RCEIL_POW2) && (fine || mxfp4) && stat != STAT_POSTROUND) {
        const int rpw = ms.rpw;
        fn = nvfp4 ? pick_multi_stat<2>(16, stat, ms.ch, ms.e) : mxfp4 ? pick_multi_stat<1>(B, stat, ms.ch, ms.e) : pick_multi_stat<0>(B, stat, ms.ch, ms.e);
        *fn_out = fn;
        *ctas_out = (P.T + (int64_t)MXN_FWD_WARPS * rpw - 1) / ((int64_t)MXN_FWD_WARPS * rpw);
        *threads_out = MXN_FWD_WARPS * kWarp;
        return fn != nullptr;
    }
    if (nvfp4 || mxfp4) fn = pick_fp4_kernel(nvfp4, nv_pair, B, stat, P.wpr, P.npass);
    else if (add) fn = B == 16 ? pick_add_mx<16, 1>(P.wpr, P.npass) : B == 32 ? pick_add_mx<32, 1>(P.wpr, P.npass) : pick_add_mx<32, 2>(P.wpr, P.npass);
    else if (e5m2) fn = B == 16 ? pick_e5m2<16, 1>(P.wpr, P.npass) : B == 32 ? pick_e5m2<32, 1>(P.wpr, P.npass) : pick_e5m2<32, 2>(P.wpr, P.npass);
    else if (has_gain) fn = B == 16 ? pick_gain_round<1>(P.round, stat, P.wpr, P.npass)
                          : B == 32 ? pick_gain_round<2>(P.round, stat, P.wpr, P.npass) : pick_gain_round<4>(P.round, stat, P.wpr, P.npass);
    else if (B == 16) fn = pick_round<16, 1>(P.round, stat, P.wpr, P.npass);
    else if (B == 32) fn = pick_round<32, 1>(P.round, stat, P.wpr, P.npass);
    else fn = pick_round<32, 2>(P.round, stat, P.wpr, P.npass);
    *fn_out = fn;
    *ctas_out = (P.T + P.rows_per_cta - 1) / P.rows_per_cta;
    *threads_out = warps * kWarp;
    return fn != nullptr;
}

cudaError_t launch_fwd(FwdParams P, int B, int stat, bool nvfp4, cudaStream_t stream)
{
    fwd_fn fn = nullptr;
    int64_t ctas = 0;
    int threads = 0;
    if (!select_fwd(P, B, stat, nvfp4, &fn, &ctas, &threads) || ctas > 0x7FFFFFFF) return cudaErrorInvalidValue;
    // Programmatic stream serialisation: the kernel may be scheduled while the previous kernel of the
    // stream drains; it does not touch memory before that kernel has completed (pdl_prologue).
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(threads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fn, P);
}

// Host-only walk over every row length the shape check admits, in every combination of block size, statistic, element
// format, gain, residual and rounding rule the entry points can ask for: counts the combinations for which no kernel is
// instantiated (a launch would be refused) and reports the first.  No device is touched.
int64_t selftest_dispatch(int64_t max_D, int64_t* first_D, int* first_case)
{
    int64_t missing = 0;
    static const uint16_t dummy = 0;
    for (int bi = 0; bi < 3; ++bi) {
        const int B = 16 << bi;
        for (int64_t D = B; D <= max_D; D += B) {
            if (!fwd_shape_supported(D, B)) continue;
            // every combination an entry point can ask for: variant 0 E4M3, 1 E4M3 with gain, 2 E5M2, 3 MXFP4,
            // 4 residual add, 5 NVFP4; the scale rounding rule varies for the E4M3 variants only
            for (int variant = 0; variant < 6; ++variant) {
                for (int stat = 0; stat < 4; ++stat) {
                    for (int round = 0; round <= MXN_ROUND_RCEIL_MAX; ++round) {
                        const bool asked =
                            variant == 0 ? (stat != STAT_POSTROUND || round == 0)
                          : variant == 1 ? (stat == STAT_RMS || stat == STAT_MX)
                          : variant == 2 ? (stat == STAT_NONE && round == 0)
                          : variant == 3 ? (stat != STAT_POSTROUND && round == 0)
                          : variant == 4 ? (stat == STAT_MX && round == 0)
                                         : (B == 16 && stat != STAT_POSTROUND && round == 0);
                        if (!asked) continue;
                        bool ok = true;
                        for (int big = 0; big < 2 && ok; ++big) {   // the choice of kernel may depend on the number of rows
                            FwdParams P = {};
                            P.T = big ? (int64_t)1 << 20 : 1;
                            P.D = (int)D;
                            P.K = (int)(D / B);
                            P.elem = variant == 2 ? ELEM_E5M2 : (variant == 3 || variant == 5) ? ELEM_E2M1 : ELEM_E4M3;
                            P.gain = variant == 1 ? &dummy : nullptr;
                            P.residual = variant == 4 ? &dummy : nullptr;
                            P.round = round;
                            fwd_fn fn = nullptr;
                            int64_t ctas = 0;
                            int threads = 0;
                            ok = select_fwd(P, B, stat, variant == 5, &fn, &ctas, &threads) && ctas >= 1 && ctas <= P.T && threads > 0;
                        }
                        if (ok) continue;
                        if (missing++ == 0) {
                            *first_D = D;
                            *first_case = ((B * 10 + variant) * 10 + stat) * 10 + round;
                        }
                    }
                }
            }
        }
    }
    return missing;
}

// ---- host side of the post-round estimator: f, its inverse and the table --------------------------
// f(sigma) = E[Y], Y = 2^floor(log2 max_i |X_i|) for B i.i.d. N(0, sigma^2) values.  Y only takes powers of two, so
// the expectation is summed over the levels it exceeds:
//     E[Y] = sum_j (2^j - 2^(j-1)) P(Y >= 2^j) = sum_j 2^(j-1) P(max_i |X_i| >= 2^j),
//     P(max >= t) = 1 - erf(u)^B = -expm1(B log1p(-erfc(u))),  u = t / (sigma sqrt 2).
// Levels far below sigma are exceeded with probability 1 to the last bit: their geometric tail is added in closed form.
static double pr_prob_max_at_least(double t, double sigma, int B)
{
    const double u = t / (sigma * 1.4142135623730951);
    return -std::expm1((double)B * std::log1p(-std::erfc(u)));
}
static double pr_expected_rounded_max(double sigma, int B)
{
    int e;
    (void)std::frexp(sigma, &e);                 // sigma in [2^(e-1), 2^e)
    const int lowest = e - 14;                   // 2^lowest < sigma 2^-12: erf(u)^B < 2^-160, the probability is exactly 1
    double total = std::ldexp(1.0, lowest - 1);  // sum over j < lowest of 2^(j-1)
    for (int j = lowest; j <= e + 8; ++j) {      // beyond 2^8 sigma the probability is below 1e-300
        const double pj = pr_prob_max_at_least(std::ldexp(1.0, j), sigma, B);
        if (pj == 0.0) break;
        total += std::ldexp(pj, j - 1);
    }
    return total;
}
// f is increasing and sigma/2 < f(sigma) < 4 sigma for the supported block sizes: a bracketing secant iteration
// (regula falsi with the Illinois modification) from that bracket
static double pr_invert(double x, int B)
{
    double a = x / 8.0, b = x * 4.0;
    double fa = pr_expected_rounded_max(a, B) - x, fb = pr_expected_rounded_max(b, B) - x;
    int side = 0;
    for (int it = 0; it < 200 && b - a > 4e-16 * b; ++it) {
        double c = (a * fb - b * fa) / (fb - fa);
        if (!(c > a && c < b)) c = 0.5 * (a + b);
        const double fc = pr_expected_rounded_max(c, B) - x;
        if (fc == 0.0) return c;
        if (fc < 0.0) {
            a = c; fa = fc;
            if (side == -1) fb *= 0.5;
            side = -1;
        } else {
            b = c; fb = fc;
            if (side == 1) fa *= 0.5;
            side = 1;
        }
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

}  // namespace mxn
