// Pieces shared by the translation units of the forward kernels: the row loader, the pre-wait L2 hint and the kernel
// pointer type of the dispatch tables.
#pragma once
#include "mxn_device.cuh"
#include "mxn_internal.h"
#include "mxn_row.cuh"

namespace mxn {

typedef void (*fwd_fn)(const FwdParams);

// The 4-bit row-group kernels (MXFP4, NVFP4 one block per lane, NVFP4 two blocks per lane) live in a translation unit of
// their own so that the two halves of the forward kernels compile side by side; nullptr when the variant does not exist.
fwd_fn pick_fp4_kernel(bool nvfp4, bool two_blocks_per_lane, int B, int stat, int wpr, int npass);

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

constexpr unsigned kFirstWaveCtas = 148 * 8;   // SMs x the most CTAs of 128 threads an SM holds at 64 registers

// One lane per row asks for the whole row in L2 before the kernel waits for its predecessor (see prefetch_l2_bulk):
// rows are multiples of 32 bytes and 32-byte aligned.
__device__ __forceinline__ void prefetch_row(const uint16_t* base, int64_t row, const FwdParams& P, int w, int lane)
{
    // only CTAs of the first wave can be resident before the previous kernel has ended; for the rest the hint is redundant
    if (w == 0 && lane == 0 && row < P.T && blockIdx.x < kFirstWaveCtas) prefetch_l2_bulk(base + row * P.D, (uint32_t)P.D * 2u);
}

}  // namespace mxn
