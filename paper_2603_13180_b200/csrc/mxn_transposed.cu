// Column-wise (transposed) MXCast: blocks of 32 consecutive TOKENS of one column, output laid out
// [D, T] - the operand layout the weight-gradient GEMM of MXNormLinear needs
// (grad W = MXCast(grad H^T) MXCast(rho~ X) gamma: the activation is re-quantised along the token axis from
// the cached X and rho~, the upstream gradient along its token axis as well).
//
// Two kernels.  The tile kernel (further down; D % 8 == 0 and a 16-byte aligned input) stages 128 tokens x 64 columns
// in shared memory, quantises column pairs from there and writes the transposed tile in whole 128-byte lines.
// The register kernel right below serves every other valid input (D % 4 == 0, 8-byte aligned): a warp owns a tile of
// 32 tokens x 128 columns; a lane owns 4 columns and walks the 32 rows (8-byte loads, a warp reads 256 contiguous
// bytes per row), so a column block's absmax needs no cross-lane traffic and its 32 codes leave as one 32-byte store
// into row c of the transposed output.  Every input byte is read once, every output byte written once.
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
        rho_l = recip_sat(__fadd_rn(P.rms[t0 + lane], P.eps));
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

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }

#ifndef MXN_TO_MINB
#define MXN_TO_MINB 7   // resident CTAs per SM aimed for (measured at [16384,4096]: 5 -> 35.1 us, 6 -> 32.9, 7 -> 32.0, 8 spills -> 40.1)
#endif

// ---- output-staged variant (D % 8 == 0, x 16-byte aligned) ------------------------------------------
// A CTA of 4 warps takes a tile of 128 tokens x 64 columns.  The 128 row segments of 128 bytes arrive with 16-byte
// cp.async copies.  Warp w quantises token block w (32 tokens) of all 64 columns exactly as the kernel above does
// (a lane owns two adjacent columns), but its 32 code bytes per column go to a shared-memory image of the OUTPUT tile
// (64 rows of the transposed matrix x 128 tokens); after one barrier the CTA writes that image row by row, eight
// threads covering the 128 contiguous bytes of one output row - whole lines instead of isolated 32-byte sectors.
// The 16-byte chunks of an image row are XOR-swizzled with the column pair index so that both the per-lane writes
// (lane l -> rows 2l, 2l+1) and the row-wise reads are bank-conflict-free.  The four scale bytes of a column (one per
// token block) leave as one 4-byte store.
constexpr int kToCols = 64, kToTokens = 128, kToThreads = 128, kToInBytes = kToTokens * kToCols * 2, kToOutBytes = kToCols * kToTokens;

template <bool PAPER, int ELEM, bool ZSPILL, bool RHO>
__global__ void __launch_bounds__(kToThreads, MXN_TO_MINB) cast_transposed_tile_kernel(const TransposedParams P)
{
    extern __shared__ __align__(128) uint8_t tile_raw[];
    __shared__ __align__(16) float rho_s[4][32];
    __shared__ __align__(16) uint8_t sb_s[kToCols][4];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t in0 = (uint32_t)__cvta_generic_to_shared(tile_raw), out0 = in0 + kToInBytes;
    const int ctile = blockIdx.x * kToCols;
    const int64_t tbase = (int64_t)token_tile_index<ZSPILL>() * kToTokens;
    {   // first-wave CTAs ask for their tile in L2 before the wait for the previous kernel: one 128-byte line per thread
        const bool first_wave = (uint64_t)token_tile_index<ZSPILL>() * gridDim.x + blockIdx.x < 148u * 9u;
        if (first_wave && tbase + tid < P.T && ctile < P.D)
            asm volatile("prefetch.global.L2 [%0];" :: "l"(P.x + (tbase + tid) * P.D + ctile) : "memory");
    }
    pdl_prologue();
    if (tbase >= P.T) return;
    const int nblocks = (int)((P.T - tbase < kToTokens ? P.T - tbase : kToTokens) >> 5);   // token blocks of this tile (T % 32 == 0)

    // 128 rows x 8 chunks of 16 bytes; thread i takes chunk i % 8 of rows i / 8 + 16 k
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int row = (tid >> 3) + 16 * k, c16 = tid & 7;
        const int col = ctile + c16 * 8;
        const uint32_t dst = in0 + (uint32_t)row * (kToCols * 2) + (uint32_t)c16 * 16;
        if (row < nblocks * 32 && col < P.D) cp_async16(dst, P.x + (tbase + row) * P.D + col);
        else asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" :: "r"(dst), "r"(0u) : "memory");
    }
    cp_async_commit();
    if (RHO) {
        float rho = 1.0f;
        if (tid < nblocks * 32) rho = recip_sat(__fadd_rn(P.rms[tbase + tid], P.eps));
        rho_s[warp][lane] = rho;
    }
    cp_async_wait<0>();
    __syncthreads();

    if (warp < nblocks) {
        const uint32_t wordaddr = in0 + (uint32_t)(warp * 32) * (kToCols * 2) + (uint32_t)lane * 4;
        uint32_t xr[32];
#pragma unroll
        for (int r = 0; r < 32; ++r) asm volatile("ld.shared.b32 %0, [%1];" : "=r"(xr[r]) : "r"(wordaddr + (uint32_t)r * (kToCols * 2)));
        uint32_t o0[8], o1[8], sb0, sb1;
        quantise_column_pair<PAPER, ELEM, RHO>(xr, rho_s[warp], P.round, o0, o1, sb0, sb1);
        // image rows 2*lane and 2*lane+1, bytes [32 warp, 32 warp + 32): chunks 2 warp and 2 warp + 1, swizzled by lane % 8
        const uint32_t r0 = out0 + (uint32_t)(2 * lane) * kToTokens, sw = (uint32_t)(lane & 7);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t chunk = ((uint32_t)(2 * warp + h) ^ sw) * 16;
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" :: "r"(r0 + chunk), "r"(o0[4 * h]), "r"(o0[4 * h + 1]), "r"(o0[4 * h + 2]), "r"(o0[4 * h + 3]) : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" :: "r"(r0 + kToTokens + chunk), "r"(o1[4 * h]), "r"(o1[4 * h + 1]), "r"(o1[4 * h + 2]), "r"(o1[4 * h + 3]) : "memory");
        }
        sb_s[2 * lane][warp] = (uint8_t)sb0;
        sb_s[2 * lane + 1][warp] = (uint8_t)sb1;
    }
    __syncthreads();

    // codes: thread i writes chunk i % 8 of image rows i / 8 + 16 k (eight threads = the 128 contiguous bytes of a row)
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int row = (tid >> 3) + 16 * k, j = tid & 7;
        const int c = ctile + row;
        if (c < P.D && j < 2 * nblocks) {
            uint32_t v[4];
            const uint32_t src = out0 + (uint32_t)row * kToTokens + (((uint32_t)j ^ (uint32_t)((row >> 1) & 7)) * 16);
            asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(src));
            st_v4(P.codes + (int64_t)c * P.T + tbase + j * 16, v);
        }
    }
    // scales: thread i < 64 writes the (up to) four scale bytes of column i
    if (tid < kToCols && ctile + tid < P.D) {
        const int64_t row = ctile + tid;
        const int k0 = (int)(tbase >> 5);          // a multiple of 4
        int64_t off;
        if (P.layout == MXN_SCALES_ROWMAJOR) {
            off = row * P.KT + k0;
        } else {
            const int rr = (int)(row & 127);
            off = ((row >> 7) * P.tiles_per_row + (k0 >> 2)) * 512 + (rr & 31) * 16 + (rr >> 5) * 4;
        }
        const uint32_t w4 = *reinterpret_cast<const uint32_t*>(sb_s[tid]);
        if (nblocks == 4 && (off & 3) == 0) {
            *reinterpret_cast<uint32_t*>(P.scales + off) = w4;
        } else {
            for (int b = 0; b < nblocks; ++b) P.scales[off + b] = (uint8_t)(w4 >> (8 * b));
        }
    }
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
    // 16-byte row chunks need D % 8 == 0 and a 16-byte aligned base (then every row start is 16-byte aligned)
    if (P.D % 8 == 0 && (reinterpret_cast<uintptr_t>(P.x) & 15) == 0) {
        const int64_t sx = (P.D + kToCols - 1) / kToCols, sy = (P.T + kToTokens - 1) / kToTokens;
        if ((sy + kMaxGridY - 1) / kMaxGridY <= 65535) {
            const bool zs = sy > kMaxGridY;
            const bool rho = P.rms != nullptr;      // without a normaliser (e.g. the upstream gradient): the cheaper column phase
            void (*kfn)(const TransposedParams);
            if (P.elem == ELEM_E5M2) kfn = zs ? cast_transposed_tile_kernel<true, 2, true, false> : cast_transposed_tile_kernel<true, 2, false, false>;
            else if (P.round == MXN_ROUND_RCEIL_POW2)
                kfn = rho ? (zs ? cast_transposed_tile_kernel<true, 0, true, true> : cast_transposed_tile_kernel<true, 0, false, true>)
                          : (zs ? cast_transposed_tile_kernel<true, 0, true, false> : cast_transposed_tile_kernel<true, 0, false, false>);
            else
                kfn = rho ? (zs ? cast_transposed_tile_kernel<false, 0, true, true> : cast_transposed_tile_kernel<false, 0, false, true>)
                          : (zs ? cast_transposed_tile_kernel<false, 0, true, false> : cast_transposed_tile_kernel<false, 0, false, false>);
            const int smem = kToInBytes + kToOutBytes;
            const cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return e;
            cfg.gridDim = token_tile_grid(sx, sy);
            cfg.blockDim = dim3(kToThreads);
            cfg.dynamicSmemBytes = smem;
            return cudaLaunchKernelEx(&cfg, kfn, P);
        }
    }
    const bool zs = gy > kMaxGridY;
    auto kfn = P.elem == ELEM_E5M2 ? (zs ? cast_transposed_kernel<true, 2, true> : cast_transposed_kernel<true, 2, false>)
               : P.round == MXN_ROUND_RCEIL_POW2 ? (zs ? cast_transposed_kernel<true, 0, true> : cast_transposed_kernel<true, 0, false>)
                                                 : (zs ? cast_transposed_kernel<false, 0, true> : cast_transposed_kernel<false, 0, false>);
    return cudaLaunchKernelEx(&cfg, kfn, P);
}

}  // namespace mxn
