// Device helpers shared by the libmxnorm kernels (sm_100a only).
//
// Arithmetic rules used throughout: every product that the contract calls "one IEEE binary32
// operation" is written with an explicit round-to-nearest intrinsic so that the compiler cannot
// contract or reassociate it; no flush-to-zero, no fast-math.
#pragma once

#include <cuda_fp4.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mxnorm.h"

namespace mxn {

constexpr int kWarp = 32;

// ---- 256-bit global memory accesses (32 bytes per lane; address 32-byte aligned) ------------
__device__ __forceinline__ void ld_v8(const void* p, uint32_t* r)
{
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "l"(p));
}
// same width through the coherent path: for buffers the kernel may also write (in-place residual update)
__device__ __forceinline__ void ld_v8_coherent(const void* p, uint32_t* r)
{
    asm volatile("ld.global.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "l"(p) : "memory");
}
__device__ __forceinline__ void st_v8(void* p, const uint32_t* r)
{
    asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void st_v4(void* p, const uint32_t* r)
{
    asm volatile("st.global.cs.v4.b32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
__device__ __forceinline__ void st_v2(void* p, const uint32_t* r)
{
    asm volatile("st.global.cs.v2.b32 [%0], {%1,%2};" :: "l"(p), "r"(r[0]), "r"(r[1]) : "memory");
}

// ---- bf16 pairs -----------------------------------------------------------------------------
// max(|a|,|b|) per bf16 half; the sign bit of the result is the xor of the signs (ignored).
__device__ __forceinline__ uint32_t absmax_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// the larger magnitude of the two halves of a bf16x2 word, as a binary32 (exact widening)
__device__ __forceinline__ float hmax_abs_to_f32(uint32_t m2)
{
    uint32_t lo = (m2 << 16) & 0x7FFF0000u, hi = m2 & 0x7FFF0000u;
    return __uint_as_float(lo > hi ? lo : hi);   // positive floats order like their bit patterns
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// a bf16 pair as two binary32 (exact widening) and the packed product with a broadcast factor:
// two IEEE round-to-nearest multiplies in one instruction
__device__ __forceinline__ float2 bf16x2_to_f32x2(uint32_t w) { return make_float2(bf16_lo(w), bf16_hi(w)); }
__device__ __forceinline__ float2 mul2(float2 a, float2 b) { return __fmul2_rn(a, b); }

// ---- element casts --------------------------------------------------------------------------
// two binary32 -> two E4M3 (RN-even, saturating to +-448); `lo` lands in the low byte
__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi)
{
    uint16_t d;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}
// four binary32 -> four E4M3 bytes in memory order
__device__ __forceinline__ uint32_t cvt_e4m3x4(float e0, float e1, float e2, float e3)
{
    uint32_t d;
    asm("{ .reg .b16 lo, hi; cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1; cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3; mov.b32 %0, {lo, hi}; }"
        : "=r"(d) : "f"(e0), "f"(e1), "f"(e2), "f"(e3));
    return d;
}
// four binary32 -> four E5M2 bytes in memory order (RN-even, saturating to +-57344)
__device__ __forceinline__ uint32_t cvt_e5m2x4(float e0, float e1, float e2, float e3)
{
    uint32_t d;
    asm("{ .reg .b16 lo, hi; cvt.rn.satfinite.e5m2x2.f32 lo, %2, %1; cvt.rn.satfinite.e5m2x2.f32 hi, %4, %3; mov.b32 %0, {lo, hi}; }"
        : "=r"(d) : "f"(e0), "f"(e1), "f"(e2), "f"(e3));
    return d;
}
// one byte per element formats: 0 = E4M3 (largest power of two 2^8), 2 = E5M2 (2^15)
template <int ELEM>
__device__ __forceinline__ uint32_t cvt_fp8x4(float e0, float e1, float e2, float e3)
{
    return ELEM == 2 ? cvt_e5m2x4(e0, e1, e2, e3) : cvt_e4m3x4(e0, e1, e2, e3);
}
// two binary32 -> two E2M1 nibbles (RN-even, saturating to +-6); `lo` lands in the low nibble
__device__ __forceinline__ uint32_t cvt_e2m1x2(float lo, float hi)
{
    return __nv_cvt_float2_to_fp4x2(make_float2(lo, hi), __NV_E2M1, cudaRoundNearest);
}
// eight binary32 -> eight E2M1 nibbles in memory order (element 0 in the low nibble of byte 0)
__device__ __forceinline__ uint32_t cvt_e2m1x8(float e0, float e1, float e2, float e3, float e4, float e5, float e6, float e7)
{
    uint32_t d;
    asm("{ .reg .b8 b0, b1, b2, b3; cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1; cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3; "
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5; cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7; mov.b32 %0, {b0, b1, b2, b3}; }"
        : "=r"(d) : "f"(e0), "f"(e1), "f"(e2), "f"(e3), "f"(e4), "f"(e5), "f"(e6), "f"(e7));
    return d;
}
// E4M3 byte (non-negative, finite) -> binary32, exact
__device__ __forceinline__ float e4m3_to_f32(uint32_t c)
{
    uint32_t ef = (c >> 3) & 0xF, mf = c & 7;
    // normal: (8+mf) * 2^(ef-10); subnormal: mf * 2^-9
    return ef ? __uint_as_float(((ef + 120u) << 23) | (mf << 20)) : (float)mf * 0.001953125f;
}

// ---- correctly rounded division by a known divisor without the division sequence ---------------------
// q = RN(a*c), r = a - q*d (exact in an FMA), q' = RN(q + r*c) with c = RN(1/d) equals RN(a/d) whenever no
// intermediate leaves the normal range.  Checked exhaustively on the device (every binary32 numerator with
// exponent in [2^-100, 2^100)) for d = 6, d = 448 and the eight E4M3 significands 1 + m/8; mxn_selftest_division
// repeats that check.  Outside the exponent window the IEEE division is used.
__device__ __forceinline__ bool in_division_window(float a)
{
    const uint32_t E = (__float_as_uint(a) >> 23) & 0xFFu;
    return E - 27u < 200u;   // 2^-100 <= |a| < 2^100
}
__device__ __forceinline__ float div_by_known(float a, float d, float c)
{
    const float q = __fmul_rn(a, c);
    const float r = __fmaf_rn(-d, q, a);
    return __fmaf_rn(r, c, q);
}
__device__ __forceinline__ float div_by_6(float a)
{
    return in_division_window(a) ? div_by_known(a, 6.0f, 0x1.555556p-3f) : __fdiv_rn(a, 6.0f);
}
// RN(1 / (1 + m/8)) for m = 0..7
__device__ __constant__ float kRcpE4M3Significand[8] = {0x1p+0f, 0x1.c71c72p-1f, 0x1.99999ap-1f, 0x1.745d18p-1f,
                                                        0x1.555556p-1f, 0x1.3b13b2p-1f, 0x1.24924ap-1f, 0x1.111112p-1f};
// a / d for d the value of the normal, non-negative E4M3 byte c (exponent field ef >= 1)
__device__ __forceinline__ float div_by_e4m3_normal(float a, uint32_t code, float d)
{
    const uint32_t ef = (code >> 3) & 0xFu, mf = code & 7u;
    // 1/d = RN(1/(1+mf/8)) * 2^-(ef-7): the power of two is exact
    const float c = __fmul_rn(kRcpE4M3Significand[mf], __uint_as_float((134u - ef) << 23));
    return div_by_known(a, d, c);
}

// ---- E8M0 block scale -----------------------------------------------------------------------
// biased exponent sb of the power-of-two scale S = 2^(sb-127) for a block whose (normalised)
// absmax is a >= 0; element format E4M3 (largest power of two 2^8, largest value 448).
__device__ __forceinline__ uint32_t e8m0_scale(float a, int round)
{
    uint32_t u = __float_as_uint(a);
    uint32_t E = u >> 23, frac = u & 0x7FFFFFu;
    if (E >= 255u) return frac ? 0u : 254u;      // not finite (outside the contract): NaN -> 0, Inf -> largest scale
    int sb;
    if (round == MXN_ROUND_RCEIL_POW2) {
        sb = (int)E + (frac != 0) - 8;           // ceil(log2 a) - 8 + 127; E == 0 (zero/subnormal) clamps to 0
    } else if (round == MXN_ROUND_FLOOR_OCP) {
        sb = (int)E - 8;                         // floor(log2 a) - 8 + 127
    } else {
        uint32_t t = __float_as_uint(__fdiv_rn(a, 448.0f));
        uint32_t Et = t >> 23;
        sb = Et ? (int)Et + ((t & 0x7FFFFFu) != 0) : (t > 0x00400000u);   // subnormal quotient: 2^-127 < t -> 1
    }
    return (uint32_t)max(sb, 0);
}
// the paper's rule only (round up a/256 to a power of two): sb = max(ceil(log2 a) - 8 + 127, 0)
template <int EMAX = 8>
__device__ __forceinline__ uint32_t e8m0_scale_rceil_pow2(float a)
{
    const uint32_t u = __float_as_uint(a);
    const uint32_t E = u >> 23;
    if (E >= 255u) return (u & 0x7FFFFFu) ? 0u : 254u;   // not finite (outside the contract)
    const int sb = (int)E + ((u & 0x7FFFFFu) != 0u) - EMAX;   // EMAX: log2 of the element format's largest power of two
    return (uint32_t)max(sb, 0);
}
// 2^(127-sb) as binary32 (sb = 254 gives the subnormal 2^-127)
__device__ __forceinline__ float inv_scale(uint32_t sb)
{
    return __uint_as_float(sb >= 254u ? 0x00400000u : ((254u - sb) << 23));
}
__device__ __forceinline__ bool is_normal_f32(float f)
{
    uint32_t E = (__float_as_uint(f) >> 23) & 0xFFu;
    return E != 0u && E != 255u;
}

// ---- normalisation factor ---------------------------------------------------------------------------
// rho = 1/den as one IEEE binary32 division; 0 for a zero denominator (a zero row stays zero) and the largest finite
// binary32 where the quotient would overflow (den < 2^-128: rows of subnormal magnitude), so that no 0 * inf = NaN can
// arise from finite input.
__device__ __forceinline__ float recip_sat(float den)
{
    return den == 0.0f ? 0.0f : fminf(__fdiv_rn(1.0f, den), 3.402823466e+38f);
}

// ---- programmatic dependent launch ----------------------------------------------------------------
// Every kernel of the library is launched with programmatic stream serialisation and starts with this
// prologue: wait until the preceding kernel of the stream has completed and its writes are visible
// (a no-op when that kernel was not launched early), then allow the following kernel to be scheduled
// while this one is still running.  Memory is only touched after the wait, so results are the same as
// with fully serialised launches; what overlaps is the launch latency and block scheduling of one
// kernel with the tail of the previous one.
// Hint: bring `bytes` (a multiple of 16, 16-byte aligned address) into L2.  A prefetch consumes no value, so it may be
// issued BEFORE griddepcontrol.wait: L2 is the point of coherence, a line prefetched early and then written by the
// previous kernel is simply updated in place, and the loads that follow the wait see the new data.  What it buys: the
// CTAs of this kernel that become resident while the previous kernel drains fill the idle DRAM with their first rows.
__device__ __forceinline__ void prefetch_l2_bulk(const void* p, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" :: "l"(p), "r"(bytes) : "memory");
}

__device__ __forceinline__ void pdl_prologue()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ---- reductions -----------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = __dadd_rn(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = __fadd_rn(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}
// barrier among the `nthreads` threads of one row group; the id is a compile-time constant (1..15)
template <int ID>
__device__ __forceinline__ void group_barrier_id(int nthreads)
{
    asm volatile("bar.sync %0, %1;" :: "n"(ID), "r"(nthreads) : "memory");
}

}  // namespace mxn
