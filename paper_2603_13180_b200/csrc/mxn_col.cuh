// Column-wise (along the tokens) quantisation of two adjacent columns over one block of 32 tokens.
#ifndef MXN_COL_CUH_
#define MXN_COL_CUH_

#include "mxn_device.cuh"
#include "mxn_internal.h"

namespace mxn {

// xr[r] = the bf16 pair (column c, column c+1) of token r of the block; rho = 32 per-token factors in shared
// memory (16-byte aligned).  y = fl32(x * rho_r); one E8M0 scale per column from max_r |y|; codes of
// fl32(y * 2^(127-sb)).  out0/out1 = the 32 code bytes of column c / c+1 in token order.
// RHO = false: no per-token factor (rho = 1, e.g. the upstream gradient): the column maxima come from packed bf16
// comparisons and every code from one product - the same results as RHO = true with factors of 1, at half the work.
template <bool PAPER, int ELEM, bool RHO = true>
__device__ __forceinline__ void quantise_column_pair(const uint32_t (&xr)[32], const float* rho, int round,
                                                     uint32_t (&out0)[8], uint32_t (&out1)[8], uint32_t& sb0, uint32_t& sb1)
{
    if constexpr (!RHO) {
        uint32_t m2 = xr[0] & 0x7FFF7FFFu;
#pragma unroll
        for (int r = 1; r < 32; ++r) m2 = absmax_bf16x2(m2, xr[r]);     // per half: max(|a|, |b|); the sign bit is not used
        const float m0 = __uint_as_float((m2 << 16) & 0x7FFF0000u), m1 = __uint_as_float(m2 & 0x7FFF0000u);
        sb0 = PAPER ? e8m0_scale_rceil_pow2<ELEM == 2 ? 15 : 8>(m0) : e8m0_scale(m0, round);
        sb1 = PAPER ? e8m0_scale_rceil_pow2<ELEM == 2 ? 15 : 8>(m1) : e8m0_scale(m1, round);
        const float2 inv = make_float2(inv_scale(sb0), inv_scale(sb1));
#pragma unroll
        for (int r = 0; r < 32; r += 4) {
            float2 q[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) q[i] = mul2(bf16x2_to_f32x2(xr[r + i]), inv);
            out0[r / 4] = cvt_fp8x4<ELEM>(q[0].x, q[1].x, q[2].x, q[3].x);
            out1[r / 4] = cvt_fp8x4<ELEM>(q[0].y, q[1].y, q[2].y, q[3].y);
        }
        return;
    }
    float m0 = 0.f, m1 = 0.f;
#pragma unroll
    for (int r = 0; r < 32; r += 4) {
        const float4 r4 = *reinterpret_cast<const float4*>(rho + r);   // broadcast read
        const float rv[4] = {r4.x, r4.y, r4.z, r4.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 y = mul2(bf16x2_to_f32x2(xr[r + i]), make_float2(rv[i], rv[i]));
            m0 = fmaxf(m0, fabsf(y.x));
            m1 = fmaxf(m1, fabsf(y.y));
        }
    }
    sb0 = PAPER ? e8m0_scale_rceil_pow2<ELEM == 2 ? 15 : 8>(m0) : e8m0_scale(m0, round);
    sb1 = PAPER ? e8m0_scale_rceil_pow2<ELEM == 2 ? 15 : 8>(m1) : e8m0_scale(m1, round);
    const float2 inv = make_float2(inv_scale(sb0), inv_scale(sb1));
#pragma unroll
    for (int r = 0; r < 32; r += 4) {
        float2 q[4];
        const float4 r4 = *reinterpret_cast<const float4*>(rho + r);
        const float rv[4] = {r4.x, r4.y, r4.z, r4.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) q[i] = mul2(mul2(bf16x2_to_f32x2(xr[r + i]), make_float2(rv[i], rv[i])), inv);
        out0[r / 4] = cvt_fp8x4<ELEM>(q[0].x, q[1].x, q[2].x, q[3].x);
        out1[r / 4] = cvt_fp8x4<ELEM>(q[0].y, q[1].y, q[2].y, q[3].y);
    }
}

// codes_t [D, T] and scales_t [D, KT] (row-major, or 128x4-tiled with the column as the row index):
// the 32 code bytes and the scale byte of columns c and c+1 for the token block starting at t0
__device__ __forceinline__ void store_column_pair(uint8_t* codes_t, uint8_t* scales_t, int64_t T, int KT, int tiles_per_row, int layout,
                                                  int c, int64_t t0, const uint32_t (&out0)[8], const uint32_t (&out1)[8],
                                                  uint32_t sb0, uint32_t sb1)
{
    const int k = (int)(t0 >> 5);
    st_v8(codes_t + (int64_t)c * T + t0, out0);
    st_v8(codes_t + (int64_t)(c + 1) * T + t0, out1);
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int64_t row = c + j;
        int64_t off;
        if (layout == MXN_SCALES_ROWMAJOR) {
            off = row * KT + k;
        } else {
            const int rr = (int)(row & 127);
            off = ((row >> 7) * tiles_per_row + (k >> 2)) * 512 + (rr & 31) * 16 + (rr >> 5) * 4 + (k & 3);
        }
        scales_t[off] = (uint8_t)(j == 0 ? sb0 : sb1);
    }
}

}  // namespace mxn
#endif  // MXN_COL_CUH_
