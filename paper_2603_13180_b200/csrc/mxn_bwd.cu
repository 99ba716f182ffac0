// Backward kernels: the RMSNorm gradient evaluated with the saved (estimated) RMS - the
// straight-through estimator of MXNorm (appendix "RMSNorm gradients").
//
//   h = g * gamma ; delta_t = (1/D) sum_d h_td x_td
//   dX_td = h_td / r_t - x_td * delta_t / r_t^3
//   dgamma_j = sum_t (x_tj / r_t) g_tj
//
// Work decomposition: a CTA owns ALL columns (thread i owns 16-byte vectors i, i+n, i+2n, ...)
// and walks over rows, two at a time, so the per-column partial sums of dgamma stay in
// registers for the whole kernel.  Each CTA writes one row of partial sums to the workspace;
// a second small kernel adds the rows in a fixed order (deterministic, no atomics).
#include <cuda_bf16.h>

#include <mutex>

#include "mxn_device.cuh"
#include "mxn_internal.h"

namespace mxn {

constexpr int kSMs = 148;          // B200
constexpr int kBwdCtasPerSM = 3;
constexpr int kBwdRows = 2;        // rows in flight per CTA iteration (1 when a thread owns 4 vectors)

__device__ __forceinline__ uint4 ldg_nc_v4(const void* p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int V, int R, bool GAIN, bool DGAIN>
__global__ void __launch_bounds__(512) bwd_kernel(const BwdParams P)
{
    __shared__ float red[R][16];
    const int tid = threadIdx.x, n = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = n >> 5;
    const int nvec = P.D >> 3;
    const float invD = __fdiv_rn(1.0f, (float)P.D);

    uint32_t gam[V][4];   // gain kept as packed bf16 pairs
    float acc[V][8];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int vi = tid + v * n;
        uint4 gw = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);   // ones
        if (GAIN && vi < nvec) gw = __ldg(reinterpret_cast<const uint4*>(P.gain) + vi);
        gam[v][0] = gw.x; gam[v][1] = gw.y; gam[v][2] = gw.z; gam[v][3] = gw.w;
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[v][j] = 0.0f;
    }

    for (int64_t row0 = (int64_t)blockIdx.x * R; row0 < P.T; row0 += (int64_t)gridDim.x * R) {
        uint4 xw[R][V], gw[R][V];
        float inv_r[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int64_t row = row0 + r;
            const bool live = row < P.T;
            inv_r[r] = live ? __fdiv_rn(1.0f, P.rms[row]) : 0.0f;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const int vi = tid + v * n;
                if (live && vi < nvec) {
                    xw[r][v] = ldg_nc_v4(reinterpret_cast<const uint4*>(P.x + row * P.D) + vi);
                    gw[r][v] = ldg_nc_v4(reinterpret_cast<const uint4*>(P.g + row * P.D) + vi);
                } else {
                    xw[r][v] = make_uint4(0, 0, 0, 0);
                    gw[r][v] = make_uint4(0, 0, 0, 0);
                }
            }
        }
        // row dots sum_d h*x and the dgamma partials
        float dot[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float d0 = 0.f, d1 = 0.f;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const uint32_t xa[4] = {xw[r][v].x, xw[r][v].y, xw[r][v].z, xw[r][v].w};
                const uint32_t ga[4] = {gw[r][v].x, gw[r][v].y, gw[r][v].z, gw[r][v].w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float x0 = bf16_lo(xa[j]), x1 = bf16_hi(xa[j]);
                    const float g0 = bf16_lo(ga[j]), g1 = bf16_hi(ga[j]);
                    const float h0 = GAIN ? g0 * bf16_lo(gam[v][j]) : g0, h1 = GAIN ? g1 * bf16_hi(gam[v][j]) : g1;
                    d0 = fmaf(h0, x0, d0);
                    d1 = fmaf(h1, x1, d1);
                    if (DGAIN) {
                        acc[v][2 * j] = fmaf(x0 * inv_r[r], g0, acc[v][2 * j]);
                        acc[v][2 * j + 1] = fmaf(x1 * inv_r[r], g1, acc[v][2 * j + 1]);
                    }
                }
            }
            dot[r] = warp_sum(d0 + d1);
        }
        if (lane == 0) {
#pragma unroll
            for (int r = 0; r < R; ++r) red[r][warp] = dot[r];
        }
        __syncthreads();
        float c1[R], c2[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float t = red[r][0];
            for (int i = 1; i < nwarps; ++i) t += red[r][i];
            const float delta = t * invD;
            c1[r] = inv_r[r];
            c2[r] = delta * inv_r[r] * inv_r[r] * inv_r[r];
        }
        __syncthreads();   // red[] is rewritten by the next iteration
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int64_t row = row0 + r;
            if (row >= P.T) continue;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const int vi = tid + v * n;
                if (vi >= nvec) continue;
                const uint32_t xa[4] = {xw[r][v].x, xw[r][v].y, xw[r][v].z, xw[r][v].w};
                const uint32_t ga[4] = {gw[r][v].x, gw[r][v].y, gw[r][v].z, gw[r][v].w};
                float o[8];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float x0 = bf16_lo(xa[j]), x1 = bf16_hi(xa[j]);
                    const float g0 = bf16_lo(ga[j]), g1 = bf16_hi(ga[j]);
                    const float h0 = GAIN ? g0 * bf16_lo(gam[v][j]) : g0, h1 = GAIN ? g1 * bf16_hi(gam[v][j]) : g1;
                    o[2 * j] = fmaf(-x0, c2[r], h0 * c1[r]);
                    o[2 * j + 1] = fmaf(-x1, c2[r], h1 * c1[r]);
                }
                if (P.dx_is_fp32) {
                    float* dp = static_cast<float*>(P.dx) + row * P.D + (int64_t)vi * 8;
                    st_v4(dp, reinterpret_cast<const uint32_t*>(o));
                    st_v4(dp + 4, reinterpret_cast<const uint32_t*>(o + 4));
                } else {
                    uint32_t pk[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) pk[j] = pack_bf16x2(o[2 * j], o[2 * j + 1]);
                    st_v4(static_cast<uint16_t*>(P.dx) + row * P.D + (int64_t)vi * 8, pk);
                }
            }
        }
    }

    if (DGAIN) {
        float* prow = P.partial + (int64_t)blockIdx.x * P.D;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int vi = tid + v * n;
            if (vi < nvec) {
                float4* q = reinterpret_cast<float4*>(prow + (int64_t)vi * 8);
                q[0] = make_float4(acc[v][0], acc[v][1], acc[v][2], acc[v][3]);
                q[1] = make_float4(acc[v][4], acc[v][5], acc[v][6], acc[v][7]);
            }
        }
    }
}

// dgain[j] = sum over the workspace rows, fixed order: 8 warps take rows w, w+8, ..., then the
// 8 warp sums are added 0..7.  One CTA per 32 columns.
__global__ void __launch_bounds__(256) bwd_dgain_reduce_kernel(const float* __restrict__ partial, float* __restrict__ dgain,
                                                              int D, int parts)
{
    __shared__ float s[8][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = blockIdx.x * 32 + lane;
    float a = 0.0f;
    if (col < D)
        for (int p = warp; p < parts; p += 8) a += partial[(int64_t)p * D + col];
    s[warp][lane] = a;
    __syncthreads();
    if (warp == 0 && col < D) {
        float t = s[0][lane];
#pragma unroll
        for (int i = 1; i < 8; ++i) t += s[i][lane];
        dgain[col] = t;
    }
}

static bool plan_bwd(int64_t D, int* threads, int* V)
{
    if (D <= 0 || D % 8 != 0) return false;
    const int64_t nvec = D / 8;
    int n = (int)(((nvec < 256 ? nvec : 256) + 31) / 32 * 32);
    int v = (int)((nvec + n - 1) / n);
    if (v > 2) {   // wide rows: more threads before more vectors per thread
        n = 512;
        v = (int)((nvec + n - 1) / n);
    }
    if (v > 4) return false;   // D <= 16384
    *threads = n;
    *V = v <= 2 ? v : 4;
    return true;
}

bool bwd_shape_supported(int64_t D)
{
    int n, v;
    return plan_bwd(D, &n, &v);
}

static int bwd_rows(int V) { return V <= 2 ? kBwdRows : 1; }

int bwd_parts(int64_t T, int64_t D)
{
    int threads, V;
    if (!plan_bwd(D, &threads, &V)) return 0;
    const int R = bwd_rows(V);
    const int64_t iters = (T + R - 1) / R;
    const int64_t cap = (int64_t)kSMs * kBwdCtasPerSM;
    return (int)(iters < cap ? (iters < 1 ? 1 : iters) : cap);
}

template <int V, int R>
static void launch_v(const BwdParams& P, int threads, cudaStream_t s)
{
    const bool gain = P.gain != nullptr, dgain = P.dgain != nullptr;
    if (gain && dgain) bwd_kernel<V, R, true, true><<<P.parts, threads, 0, s>>>(P);
    else if (gain) bwd_kernel<V, R, true, false><<<P.parts, threads, 0, s>>>(P);
    else if (dgain) bwd_kernel<V, R, false, true><<<P.parts, threads, 0, s>>>(P);
    else bwd_kernel<V, R, false, false><<<P.parts, threads, 0, s>>>(P);
}

cudaError_t launch_bwd(BwdParams P, cudaStream_t stream)
{
    int threads, V;
    if (!plan_bwd(P.D, &threads, &V)) return cudaErrorInvalidValue;
    switch (V) {
        case 1: launch_v<1, kBwdRows>(P, threads, stream); break;
        case 2: launch_v<2, kBwdRows>(P, threads, stream); break;
        default: launch_v<4, 1>(P, threads, stream); break;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (P.dgain != nullptr) {
        bwd_dgain_reduce_kernel<<<(P.D + 31) / 32, 256, 0, stream>>>(P.partial, P.dgain, P.D, P.parts);
        e = cudaGetLastError();
    }
    return e;
}

}  // namespace mxn

// ---- backward without any caller-provided scratch -------------------------------------------------
//
// Some callers of mxnorm_bwd cannot hand over a workspace because they cannot allocate device memory
// at the point of the call: code running inside a framework's static memory plan, a plug-in that
// only receives the tensors of the op, or a host thread that must not touch the allocator while
// another stream is being captured.  For them the partial sums of dgamma live in a fixed array that
// is part of this library's device image.  Every GPU that loads the library reserves it until the
// process exits, so it is kept modest: 2 Mi floats = 8 MiB.
namespace {

constexpr size_t kNoAllocScratchFloats = size_t(2) << 20;
static __device__ __align__(256) float g_noalloc_scratch[kNoAllocScratchFloats];

// In host code the name g_noalloc_scratch is only a handle for the symbol; the device address has
// to be asked for once per device, with that device current.
constexpr int kNoAllocMaxDevices = 64;
float* g_noalloc_ptr[kNoAllocMaxDevices] = {};
std::mutex g_noalloc_mutex;

cudaError_t noalloc_scratch_for_current_device(float** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kNoAllocMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (g_noalloc_ptr[dev] == nullptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        if (p == nullptr) return cudaErrorInvalidSymbol;
        g_noalloc_ptr[dev] = static_cast<float*>(p);
    }
    *out = g_noalloc_ptr[dev];
    return cudaSuccess;
}

inline bool noalloc_misaligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }

}  // namespace

extern "C" size_t mxnorm_bwd_noalloc_max_scratch_bytes(void) { return kNoAllocScratchFloats * sizeof(float); }

extern "C" mxn_status mxnorm_bwd_noalloc(const void* x_bf16, const void* grad_out_bf16, const void* gain_bf16_or_null,
                                         const float* rms, int64_t T, int64_t D, void* dx, int dx_is_fp32,
                                         float* dgain_f32_or_null, void* cuda_stream)
{
    if (T < 0 || D <= 0 || !mxn::bwd_shape_supported(D)) return MXN_ERR_SHAPE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (T == 0) {
        if (dgain_f32_or_null != nullptr &&
            cudaMemsetAsync(dgain_f32_or_null, 0, sizeof(float) * (size_t)D, s) != cudaSuccess)
            return MXN_ERR_CUDA;
        return MXN_OK;
    }
    if (x_bf16 == nullptr || grad_out_bf16 == nullptr || rms == nullptr || dx == nullptr) return MXN_ERR_NULL;
    if (noalloc_misaligned(x_bf16, 16) || noalloc_misaligned(grad_out_bf16, 16) || noalloc_misaligned(dx, 16) ||
        noalloc_misaligned(rms, 4) || (gain_bf16_or_null != nullptr && noalloc_misaligned(gain_bf16_or_null, 16)) ||
        (dgain_f32_or_null != nullptr && noalloc_misaligned(dgain_f32_or_null, 16)))
        return MXN_ERR_ALIGN;
    const int parts = mxn::bwd_parts(T, D);
    // the same launch as mxnorm_bwd needs parts * D floats of scratch: refuse what does not fit
    if (dgain_f32_or_null != nullptr && (size_t)parts * (size_t)D > kNoAllocScratchFloats) return MXN_ERR_TOO_LARGE;
    float* scratch = nullptr;
    if (dgain_f32_or_null != nullptr && noalloc_scratch_for_current_device(&scratch) != cudaSuccess)
        return MXN_ERR_CUDA;
    mxn::BwdParams P{};
    P.x = static_cast<const uint16_t*>(x_bf16);
    P.g = static_cast<const uint16_t*>(grad_out_bf16);
    P.gain = static_cast<const uint16_t*>(gain_bf16_or_null);
    P.rms = rms;
    P.dx = dx;
    P.dgain = dgain_f32_or_null;
    P.partial = scratch;   // every one of the `parts` rows is fully rewritten by its CTA: nothing to clear
    P.T = T;
    P.D = (int)D;
    P.dx_is_fp32 = dx_is_fp32 != 0;
    P.parts = parts;
    return mxn::launch_bwd(P, s) == cudaSuccess ? MXN_OK : MXN_ERR_CUDA;
}
