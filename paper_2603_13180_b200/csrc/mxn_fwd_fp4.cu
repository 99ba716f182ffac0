// Forward kernels of the 4-bit formats with one row per row group: MXFP4 (E2M1 codes, E8M0 scales) and NVFP4 (E2M1
// codes, E4M3 scales of 16-element blocks; one or two blocks per lane).  Same work decomposition as the E4M3 kernels.
#include "mxn_fwd_common.cuh"

namespace mxn {

// E2M1 codes with E8M0 scales (MXFP4): no gain, the paper's rounding rule
template <int B, int NPASS, int WPR, int STAT, int LPB = 1>
__global__ void __launch_bounds__(cta_warps(WPR) * 32, fwd_min_ctas(WPR)) fwd_mxfp4_kernel(const FwdParams P)
{
    __shared__ double red[WPR > 1 ? cta_warps(WPR) : 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int group = warp / WPR, w = warp - group * WPR;
    const int64_t row = (int64_t)blockIdx.x * rows_per_cta(WPR) + group;
    prefetch_row(P.x, row, P, w, lane);
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
__global__ void __launch_bounds__(cta_warps(WPR) * 32, fwd_min_ctas(WPR)) fwd_nvfp4_kernel(const FwdParams P)
{
    __shared__ double red[WPR > 1 ? cta_warps(WPR) : 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int group = warp / WPR, w = warp - group * WPR;
    const int64_t row = (int64_t)blockIdx.x * rows_per_cta(WPR) + group;
    prefetch_row(P.x, row, P, w, lane);
    pdl_prologue();
    if (row >= P.T) return;

    uint32_t xr[NPASS][8];
    float m[NPASS];
    load_row_direct<16, NPASS>(xr, P.x + row * P.D, P.chunks, WPR, w, lane);
    double stat = block_stats<16, NPASS, STAT>(xr, m, P.p);
    if (STAT == STAT_RMS) forget_unpacked<NPASS, 8>(xr);
    float r = 1.0f, rho = 1.0f;
    if (STAT != STAT_NONE) {
        stat = group_sum<WPR>(stat, group, w, red);
        finish_stat<STAT>(stat, P, r, rho);
        if (P.rms_out != nullptr && w == 0 && lane == 0) P.rms_out[row] = r;
    }
    quantise_store_nvfp4<NPASS, WPR>(xr, m, rho, P, row, w, lane);
}

// NVFP4 with two blocks per lane and pass (rows of an even number of blocks): see quantise_pair_nvfp4
// (four-warp CTAs at 64 registers, 8 CTAs per SM: 26.5 -> 26.0 us at [16384,4096] against 66 registers, 7 CTAs)
template <int NPASS, int WPR, int STAT>
__global__ void __launch_bounds__(cta_warps(WPR) * 32, fwd_min_ctas(WPR)) fwd_nvfp4_pair_kernel(const FwdParams P)
{
    __shared__ double red[WPR > 1 ? cta_warps(WPR) : 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int group = warp / WPR, w = warp - group * WPR;
    const int64_t row = (int64_t)blockIdx.x * rows_per_cta(WPR) + group;
    prefetch_row(P.x, row, P, w, lane);
    pdl_prologue();
    if (row >= P.T) return;

    uint32_t xr[NPASS][16];
    float m0[NPASS], m1[NPASS];
    load_row_direct<32, NPASS>(xr, P.x + row * P.D, P.chunks, WPR, w, lane);
    double stat = 0.0;
    float2 ssa = make_float2(0.f, 0.f), ssb = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < NPASS; ++i) {
        uint32_t ma = absmax_bf16x2(xr[i][0], xr[i][1]), mb = absmax_bf16x2(xr[i][8], xr[i][9]);
#pragma unroll
        for (int j = 2; j < 8; ++j) {
            ma = absmax_bf16x2(ma, xr[i][j]);
            mb = absmax_bf16x2(mb, xr[i][8 + j]);
        }
        m0[i] = hmax_abs_to_f32(ma);
        m1[i] = hmax_abs_to_f32(mb);
        if (STAT == STAT_MX) {
            const double d0 = (double)m0[i], d1 = (double)m1[i];
            stat = P.p == 2 ? __fma_rn(d1, d1, __fma_rn(d0, d0, stat)) : __dadd_rn(__dadd_rn(stat, d0), d1);
        }
        if (STAT == STAT_RMS) {
#pragma unroll
            for (int j = 0; j < 16; j += 2) {
                const float2 a = bf16x2_to_f32x2(xr[i][j]), b = bf16x2_to_f32x2(xr[i][j + 1]);
                ssa = __ffma2_rn(a, a, ssa);
                ssb = __ffma2_rn(b, b, ssb);
            }
        }
    }
    if (STAT == STAT_RMS) {
        stat = (double)ssa.x + (double)ssa.y + ((double)ssb.x + (double)ssb.y);
        forget_unpacked<NPASS, 16>(xr);
    }
    float r = 1.0f, rho = 1.0f;
    if (STAT != STAT_NONE) {
        stat = group_sum<WPR>(stat, group, w, red);
        finish_stat<STAT>(stat, P, r, rho);
        if (P.rms_out != nullptr && w == 0 && lane == 0) P.rms_out[row] = r;
    }
    quantise_store_nvfp4_pair<NPASS, WPR>(xr, m0, m1, rho, P, row, w, lane);
}

// ---- dispatch ---------------------------------------------------------------------------------
template <int B, int LPB, int NPASS, int STAT>
static fwd_fn mxfp4_by_wpr(int wpr)
{
    switch (wpr) {
        case 1: return fwd_mxfp4_kernel<B, NPASS, 1, STAT, LPB>;
        case 2: return fwd_mxfp4_kernel<B, NPASS, 2, STAT, LPB>;
        case 3: return fwd_mxfp4_kernel<B, NPASS, 3, STAT, LPB>;
        case 4: return fwd_mxfp4_kernel<B, NPASS, 4, STAT, LPB>;
        case 5: return fwd_mxfp4_kernel<B, NPASS, 5, STAT, LPB>;
        case 6: return fwd_mxfp4_kernel<B, NPASS, 6, STAT, LPB>;
        case 7: return fwd_mxfp4_kernel<B, NPASS, 7, STAT, LPB>;
        case 8: return fwd_mxfp4_kernel<B, NPASS, 8, STAT, LPB>;
        case 16: return fwd_mxfp4_kernel<B, NPASS, 16, STAT, LPB>;
        default: return nullptr;
    }
}

// the same set of (warps per row, passes) as the E4M3 headline kernels: every count in kFineWpr with the full pass
// count, half of it (four-pass kernels) or one pass; one warp per row with any pass count
template <int B, int LPB, int STAT>
static fwd_fn pick_mxfp4(int wpr, int npass)
{
    constexpr int MAXP = MXN_FWD_MAX_ELEMS / B;
    if (wpr > 1) {
        if (npass == MAXP) return mxfp4_by_wpr<B, LPB, MAXP, STAT>(wpr);
        if (MAXP >= 4 && npass == MAXP / 2) return mxfp4_by_wpr<B, LPB, (MAXP >= 4 ? MAXP / 2 : 1), STAT>(wpr);
        if (npass == 1) return mxfp4_by_wpr<B, LPB, 1, STAT>(wpr);
        return nullptr;
    }
    switch (npass) {
        case 1: return fwd_mxfp4_kernel<B, 1, 1, STAT, LPB>;
        case 2: return fwd_mxfp4_kernel<B, (MAXP >= 2 ? 2 : MAXP), 1, STAT, LPB>;
        case 3: return fwd_mxfp4_kernel<B, (MAXP >= 3 ? 3 : MAXP), 1, STAT, LPB>;
        default: return fwd_mxfp4_kernel<B, MAXP, 1, STAT, LPB>;
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

template <int NPASS, int STAT>
static fwd_fn nvfp4_pair_by_wpr(int wpr)
{
    switch (wpr) {
        case 1: return fwd_nvfp4_pair_kernel<NPASS, 1, STAT>;
        case 2: return fwd_nvfp4_pair_kernel<NPASS, 2, STAT>;
        case 3: return fwd_nvfp4_pair_kernel<NPASS, 3, STAT>;
        case 4: return fwd_nvfp4_pair_kernel<NPASS, 4, STAT>;
        case 5: return fwd_nvfp4_pair_kernel<NPASS, 5, STAT>;
        case 6: return fwd_nvfp4_pair_kernel<NPASS, 6, STAT>;
        case 7: return fwd_nvfp4_pair_kernel<NPASS, 7, STAT>;
        case 8: return fwd_nvfp4_pair_kernel<NPASS, 8, STAT>;
        case 16: return fwd_nvfp4_pair_kernel<NPASS, 16, STAT>;
        default: return nullptr;
    }
}

template <int STAT>
static fwd_fn pick_nvfp4_pair(int wpr, int npass)
{
    return npass == 2 ? nvfp4_pair_by_wpr<2, STAT>(wpr) : npass == 1 ? nvfp4_pair_by_wpr<1, STAT>(wpr) : nullptr;
}
fwd_fn pick_fp4_kernel(bool nvfp4, bool two_blocks_per_lane, int B, int stat, int wpr, int npass)
{
    if (nvfp4 && two_blocks_per_lane)
        return stat == STAT_RMS ? pick_nvfp4_pair<STAT_RMS>(wpr, npass) : stat == STAT_NONE ? pick_nvfp4_pair<STAT_NONE>(wpr, npass) : pick_nvfp4_pair<STAT_MX>(wpr, npass);
    if (nvfp4) return stat == STAT_RMS ? pick_nvfp4<STAT_RMS>(wpr, npass) : stat == STAT_NONE ? pick_nvfp4<STAT_NONE>(wpr, npass) : pick_nvfp4<STAT_MX>(wpr, npass);
    return B == 16 ? pick_mxfp4_stat<16, 1>(stat, wpr, npass) : B == 32 ? pick_mxfp4_stat<32, 1>(stat, wpr, npass) : pick_mxfp4_stat<32, 2>(stat, wpr, npass);
}

}  // namespace mxn
