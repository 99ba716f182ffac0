// Column-wise (transposed) MXCast: blocks of 32 consecutive TOKENS of one column, output laid out
// [D, T] - the operand layout the weight-gradient GEMM of MXNormLinear needs
// (grad W = MXCast(grad H^T) MXCast(rho~ X) gamma: the activation is re-quantised along the token axis from
// the cached X and rho~, the upstream gradient along its token axis as well).
//
// Work decomposition: a warp owns a tile of 32 tokens x 128 columns; a lane owns 4 columns and walks the
// 32 rows (8-byte loads, a warp reads 256 contiguous bytes per row), so a column block's absmax needs no
// cross-lane traffic and its 32 codes leave as one 32-byte store into row c of the transposed output.
// The 4 warps of a CTA take 4 consecutive token tiles of the same columns, so each output row receives
// 128 contiguous bytes per CTA.  Every input byte is read once, every output byte written once.
#include "mxn_device.cuh"
#include "mxn_internal.h"
#include "mxn_col.cuh"

namespace mxn {

// Token tiles are spread over grid dimensions y and z (y alone is limited to 65535 tiles); ZSPILL selects the kernels
// that read blockIdx.z (the common case, z = 1, keeps the two-dimensional code: measured 1.5 % faster at [16384,4096])
constexpr unsigned kMaxGridY = 65535;
template <bool ZSPILL>
__device__ __forceinline__ unsigned token_tile_index() { return ZSPILL ? blockIdx.z * kMaxGridY + blockIdx.y : blockIdx.y; }
static dim3 token_tile_grid(int64_t col_tiles, int64_t token_tiles)
{
    const int64_t z = (token_tiles + kMaxGridY - 1) / kMaxGridY;
    return dim3((unsigned)col_tiles, (unsigned)(z > 1 ? kMaxGridY : token_tiles), (unsigned)z);
}


__device__ __forceinline__ uint2 ld_v2(const void* p)
{
    uint2 r;
    asm volatile("ld.global.nc.L1::no_allocate.v2.b32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(p));
    return r;
}

#ifndef MXN_TR_CPL
#define MXN_TR_CPL 4   // columns per lane (2 or 4); measured at [16384,4096]: 4 -> 41.9 us, 2 -> 45.7 us (narrower loads lose more than the extra warps gain)
#endif
constexpr int kTrCpl = MXN_TR_CPL;
constexpr int kTrTileCols = 32 * kTrCpl;

template <bool PAPER, int ELEM, bool ZSPILL>
__global__ void __launch_bounds__(128) cast_transposed_kernel(const TransposedParams P)
{
    constexpr int CPL = kTrCpl, WORDS = CPL / 2;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t t0 = ((int64_t)token_tile_index<ZSPILL>() * 4 + warp) * 32;
    const int c0 = blockIdx.x * kTrTileCols + lane * CPL;
    pdl_prologue();
    if (t0 >= P.T) return;
    const bool live = c0 < P.D;   // D % 4 == 0: a lane's columns are all inside or all outside

    // rho of row t0 + lane
    float rho_l = 1.0f;
    if (P.rms != nullptr) {
        const float den = __fadd_rn(P.rms[t0 + lane], P.eps);
        rho_l = den == 0.0f ? 0.0f : __fdiv_rn(1.0f, den);
    }
    uint32_t xr[32][WORDS];
#pragma unroll
    for (int r = 0; r < 32; ++r) {
        const uint16_t* p = P.x + (t0 + r) * P.D + c0;
        if (!live) {
#pragma unroll
            for (int j = 0; j < WORDS; ++j) xr[r][j] = 0u;
        } else if (WORDS == 2) {
            const uint2 v = ld_v2(p);
            xr[r][0] = v.x;
            xr[r][WORDS - 1] = v.y;
        } else {
            asm volatile("ld.global.nc.L1::no_allocate.b32 %0, [%1];" : "=r"(xr[r][0]) : "l"(p));
        }
    }

    // pass 1: y = fl32(x * rho_t); column absmaxes over the 32 tokens
    float mm[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) mm[c] = 0.0f;
#pragma unroll
    for (int r = 0; r < 32; ++r) {
        const float rho = __shfl_sync(0xFFFFFFFFu, rho_l, r);
        const float2 rr = make_float2(rho, rho);
#pragma unroll
        for (int j = 0; j < WORDS; ++j) {
            const float2 y = mul2(bf16x2_to_f32x2(xr[r][j]), rr);
            mm[2 * j] = fmaxf(mm[2 * j], fabsf(y.x));
            mm[2 * j + 1] = fmaxf(mm[2 * j + 1], fabsf(y.y));
        }
    }
    uint32_t sb[CPL];
    float2 inv[WORDS];
#pragma unroll
    for (int j = 0; j < WORDS; ++j) {
        sb[2 * j] = PAPER ? e8m0_scale_rceil_pow2<ELEM == 2 ? 15 : 8>(mm[2 * j]) : e8m0_scale(mm[2 * j], P.round);
        sb[2 * j + 1] = PAPER ? e8m0_scale_rceil_pow2<ELEM == 2 ? 15 : 8>(mm[2 * j + 1]) : e8m0_scale(mm[2 * j + 1], P.round);
        inv[j] = make_float2(inv_scale(sb[2 * j]), inv_scale(sb[2 * j + 1]));
    }

    // pass 2: q = y * 2^(127-sb); four tokens of one column make one output word
    uint32_t out[CPL][8];
#pragma unroll
    for (int r = 0; r < 32; r += 4) {
        float2 q[4][WORDS];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float rho = __shfl_sync(0xFFFFFFFFu, rho_l, r + i);
            const float2 rr = make_float2(rho, rho);
#pragma unroll
            for (int j = 0; j < WORDS; ++j) q[i][j] = mul2(mul2(bf16x2_to_f32x2(xr[r + i][j]), rr), inv[j]);
        }
#pragma unroll
        for (int j = 0; j < WORDS; ++j) {
            out[2 * j][r / 4] = cvt_fp8x4<ELEM>(q[0][j].x, q[1][j].x, q[2][j].x, q[3][j].x);
            out[2 * j + 1][r / 4] = cvt_fp8x4<ELEM>(q[0][j].y, q[1][j].y, q[2][j].y, q[3][j].y);
        }
    }
    if (!live) return;
    const int k = (int)(t0 >> 5);
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
        st_v8(P.codes + (int64_t)(c0 + c) * P.T + t0, out[c]);
        const int64_t row = c0 + c;
        int64_t off;
        if (P.layout == MXN_SCALES_ROWMAJOR) {
            off = row * P.KT + k;
        } else {
            const int rr = (int)(row & 127);
            off = ((row >> 7) * P.tiles_per_row + (k >> 2)) * 512 + (rr & 31) * 16 + (rr >> 5) * 4 + (k & 3);
        }
        P.scales[off] = (uint8_t)sb[c];
    }
}

// ---- shared-memory staged variant (D % 8 == 0) ----------------------------------------------------
// A CTA of 2 warps takes a tile of 32 tokens x 128 columns: the 32 row segments of 256 bytes arrive with
// 16-byte cp.async copies (fully coalesced, no registers held while they fly), then a lane owns two
// adjacent columns and walks the 32 rows through shared memory (consecutive lanes read consecutive words:
// conflict-free).  A CTA processes MXN_TR_TPC consecutive token tiles of the same columns with two stages,
// so the next tile streams in while the current one is quantised.
#ifndef MXN_TR_TPC
#define MXN_TR_TPC 1   // token tiles per CTA (measured at [16384,4096]: 1 -> 39.0 us, 2 -> 49.2, 4 -> 47.5)
#endif
#ifndef MXN_TR_MINB
#define MXN_TR_MINB 12
#endif
constexpr int kTsStages = MXN_TR_TPC > 1 ? 2 : 1;
#ifndef MXN_TR_COLS
#define MXN_TR_COLS 128   // columns per CTA tile, 64 per warp (measured at [16384,4096]: 64 -> 36.4 us, 128 -> 34.1, 256 -> 36.0, 512 -> 40.7, 1024 -> 54.2)
#endif
constexpr int kTsCols = MXN_TR_COLS, kTsThreads = kTsCols / 2, kTsRowBytes = kTsCols * 2, kTsStageBytes = 32 * kTsRowBytes,
              kTsTpc = MXN_TR_TPC, kTsChunksPerRow = kTsRowBytes / 16, kTsChunksPerThread = 32 * kTsChunksPerRow / kTsThreads;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }

template <bool PAPER, int ELEM, bool ZSPILL>
__global__ void __launch_bounds__(kTsThreads, MXN_TR_MINB) cast_transposed_smem_kernel(const TransposedParams P)
{
    extern __shared__ __align__(128) uint8_t tile_raw[];
    __shared__ __align__(16) float rho_s[2][32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t tile0 = (uint32_t)__cvta_generic_to_shared(tile_raw);
    const int ctile = blockIdx.x * kTsCols;                  // first column of the CTA's tile
    const int64_t tbase = (int64_t)token_tile_index<ZSPILL>() * kTsTpc * 32;   // first token of the CTA
    {   // the first tile into L2 before the wait for the previous kernel (a hint: see prefetch_l2_bulk): one 128-byte line per thread
        const int row = tid / (kTsRowBytes / 128), part = tid % (kTsRowBytes / 128);
        const bool first_wave = (uint64_t)token_tile_index<ZSPILL>() * gridDim.x < 148u * 16u;   // later CTAs start after the wait is over
        if (first_wave && row < 32 && tbase + row < P.T && ctile + part * 64 < P.D)
            asm volatile("prefetch.global.L2 [%0];" :: "l"(P.x + (tbase + row) * P.D + ctile + part * 64) : "memory");
    }
    pdl_prologue();

    auto issue = [&](int tt) {
        const int64_t t0 = tbase + (int64_t)tt * 32;
        const uint32_t stage = tile0 + (uint32_t)(tt & 1) * kTsStageBytes;
        if (t0 < P.T) {
#pragma unroll
            for (int i = 0; i < kTsChunksPerThread; ++i) {
                const int id = i * kTsThreads + tid, row = id / kTsChunksPerRow, c16 = id % kTsChunksPerRow;
                const int col = ctile + c16 * 8;
                const uint32_t dst = stage + (uint32_t)row * kTsRowBytes + (uint32_t)c16 * 16;
                if (col < P.D) cp_async16(dst, P.x + (t0 + row) * P.D + col);
                else asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" :: "r"(dst), "r"(0u) : "memory");
            }
            if (tid < 32) {
                float rho = 1.0f;
                if (P.rms != nullptr) {
                    const float den = __fadd_rn(P.rms[t0 + tid], P.eps);
                    rho = den == 0.0f ? 0.0f : __fdiv_rn(1.0f, den);
                }
                rho_s[tt & 1][tid] = rho;
            }
        }
        cp_async_commit();
    };

    issue(0);
#pragma unroll 1
    for (int tt = 0; tt < kTsTpc; ++tt) {
        const int64_t t0 = tbase + (int64_t)tt * 32;
        if (t0 >= P.T) break;                       // uniform over the CTA
        if (tt + 1 < kTsTpc) issue(tt + 1);
        else cp_async_commit();                     // keeps the group count uniform
        cp_async_wait<1>();
        __syncthreads();

        const uint32_t stage = tile0 + (uint32_t)(tt & 1) * kTsStageBytes;
        const float* rho = rho_s[tt & 1];
        const uint32_t wordaddr = stage + (uint32_t)(warp * 32 + lane) * 4;
        uint32_t xr[32];
#pragma unroll
        for (int r = 0; r < 32; ++r) asm volatile("ld.shared.b32 %0, [%1];" : "=r"(xr[r]) : "r"(wordaddr + (uint32_t)r * kTsRowBytes));

        uint32_t out0[8], out1[8], sb0, sb1;
        quantise_column_pair<PAPER, ELEM>(xr, rho, P.round, out0, out1, sb0, sb1);
        const int c = ctile + (warp * 32 + lane) * 2;
        if (c < P.D) store_column_pair(P.codes, P.scales, P.T, P.KT, P.tiles_per_row, P.layout, c, t0, out0, out1, sb0, sb1);
        __syncthreads();   // the stage may be refilled by the next issue()
    }
    cp_async_wait<0>();
}

cudaError_t launch_cast_transposed(TransposedParams P, cudaStream_t stream)
{
    P.KT = (int)(P.T / 32);
    P.tiles_per_row = (P.KT + 3) / 4;
    // grid: x = column tiles, (y, z) = token tiles (more than kMaxGridY of them spill into z; CTAs past the end leave at once)
    const int64_t gx = (P.D + kTrTileCols - 1) / kTrTileCols, gy = (P.T + 127) / 128;
    if (gx > 0x7FFFFFFF || (gy + kMaxGridY - 1) / kMaxGridY > 65535) return cudaErrorInvalidValue;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = token_tile_grid(gx, gy);
    cfg.blockDim = dim3(128);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
#ifndef MXN_TR_NO_SMEM
    if (P.D % 8 == 0) {   // 16-byte row chunks: the shared-memory staged kernel
        const int64_t sx = (P.D + kTsCols - 1) / kTsCols, sy = (P.T / 32 + kTsTpc - 1) / kTsTpc;
        if ((sy + kMaxGridY - 1) / kMaxGridY <= 65535) {
            const bool zs = sy > kMaxGridY;
            auto kfn = P.elem == ELEM_E5M2 ? (zs ? cast_transposed_smem_kernel<true, 2, true> : cast_transposed_smem_kernel<true, 2, false>)
                       : P.round == MXN_ROUND_RCEIL_POW2 ? (zs ? cast_transposed_smem_kernel<true, 0, true> : cast_transposed_smem_kernel<true, 0, false>)
                                                         : (zs ? cast_transposed_smem_kernel<false, 0, true> : cast_transposed_smem_kernel<false, 0, false>);
            const int smem = kTsStages * kTsStageBytes;
            const cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return e;
            cfg.gridDim = token_tile_grid(sx, sy);
            cfg.blockDim = dim3(kTsThreads);
            cfg.dynamicSmemBytes = smem;
            return cudaLaunchKernelEx(&cfg, kfn, P);
        }
    }
#endif
    const bool zs = gy > kMaxGridY;
    auto kfn = P.elem == ELEM_E5M2 ? (zs ? cast_transposed_kernel<true, 2, true> : cast_transposed_kernel<true, 2, false>)
               : P.round == MXN_ROUND_RCEIL_POW2 ? (zs ? cast_transposed_kernel<true, 0, true> : cast_transposed_kernel<true, 0, false>)
                                                 : (zs ? cast_transposed_kernel<false, 0, true> : cast_transposed_kernel<false, 0, false>);
    return cudaLaunchKernelEx(&cfg, kfn, P);
}

}  // namespace mxn
