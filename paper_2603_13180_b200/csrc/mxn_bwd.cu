// Backward kernels: the RMSNorm gradient evaluated with the saved (estimated) RMS - the
// straight-through estimator of MXNorm (appendix "RMSNorm gradients").
//
//   h = g * gamma ; delta_t = (1/D) sum_d h_td x_td
//   dX_td = h_td / r_t - x_td * delta_t / r_t^3
//   dgamma_j = sum_t (x_tj / r_t) g_tj
//
// Work decomposition: a CTA owns ALL columns (thread i owns 16-byte vectors i, i+n, i+2n, ...)
// and walks over rows blockIdx, blockIdx + grid, ..., so the per-column partial sums of dgamma stay
// in registers for the whole kernel.  Because the CTA is resident for many rows, the rows are fed
// through a ring of shared-memory stages: one thread asks the bulk-copy engine for the x and g rows
// of iteration i+STAGES (two instructions per row, completion signalled on an mbarrier) while the
// CTA works on iteration i, which keeps STAGES rows per CTA in flight.  Each thread reads back only
// the vectors it owns.  One __syncthreads per row (the row dot product) doubles as the "stage is
// free" signal.  Each CTA writes one row of partial sums to the workspace; a second small kernel
// adds the rows in a fixed order (deterministic, no atomics).
//
// Every wait on an mbarrier is bounded; if one runs out the CTA stops and a device-side counter is
// raised (mxn_device_timeouts()).
#include <cuda_bf16.h>

#include <mutex>

#include "mxn_device.cuh"
#include "mxn_internal.h"

namespace mxn {

constexpr int kSMs = 148;          // B200

__device__ unsigned int g_bwd_timeouts = 0;

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// false when the barrier did not complete within `limit` polls (the default is of the order of a second)
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit = 1u << 20)
{
    for (uint32_t spin = 0; spin < limit; ++spin)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// global -> shared bulk copy (no multicast); addresses 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ uint4 lds_v4(uint32_t addr)
{
    uint4 r;
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}

constexpr int kBwdMaxStages = 8;

#ifndef MXN_BWD_THREADS
#define MXN_BWD_THREADS 256      // threads per CTA for rows that need more than one vector per thread
#endif
#ifndef MXN_BWD_CTAS
#define MXN_BWD_CTAS 2           // resident CTAs per SM the register allocator and the ring size aim for
#endif

// resident CTAs per SM the register allocator is asked to make room for: CTAs of at most 192 threads (short rows, or
// one vector per thread) need few registers and little shared memory, and only more CTAs per SM give short rows enough
// rows in flight
__host__ __device__ constexpr int bwd_ctas_per_sm(int V, int NT) { return NT > MXN_BWD_THREADS ? 1 : (V == 1 || NT <= 192) ? 3 : MXN_BWD_CTAS; }

template <int V, int NT, bool GAIN, bool DGAIN>
__global__ void __launch_bounds__(NT, bwd_ctas_per_sm(V, NT)) bwd_kernel(const BwdParams P)
{
    // four vectors per thread with gain and gain gradient do not fit 128 registers if t = g/r*gamma is kept between the
    // two phases of a row: that variant recomputes it (the same operations, hence the same bits)
    constexpr bool KEEP_T = !(V == 4 && GAIN && DGAIN);
    extern __shared__ __align__(128) uint8_t ring_raw[];
    __shared__ uint64_t full[kBwdMaxStages];
    __shared__ float red[2][16];
    __shared__ int abort_flag;

    const int tid = threadIdx.x, n = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = n >> 5;
    const int nvec = P.D >> 3;
    const int stages = P.stages;
    const uint32_t row_bytes = (uint32_t)P.D * 2u, half = (uint32_t)P.stage_bytes / 2u;
    const uint32_t ring = smem_u32(ring_raw), bar0 = smem_u32(full);
    const float invD = __fdiv_rn(1.0f, (float)P.D);
    const int64_t stride = gridDim.x;

    if (tid < 2 * stages) {   // the first ring fill into L2 before the wait for the previous kernel (see prefetch_l2_bulk)
        const int64_t row = (int64_t)blockIdx.x + (tid >> 1) * stride;
        if (row < P.T) prefetch_l2_bulk(((tid & 1) ? P.g : P.x) + row * P.D, row_bytes);
    }
    pdl_prologue();
    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < stages; ++s) mbar_init(bar0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        for (int s = 0; s < stages; ++s) {
            const int64_t row = (int64_t)blockIdx.x + s * stride;
            if (row < P.T) {
                mbar_expect_tx(bar0 + 8 * s, 2 * row_bytes);
                bulk_load(ring + s * P.stage_bytes, P.x + row * P.D, row_bytes, bar0 + 8 * s);
                bulk_load(ring + s * P.stage_bytes + half, P.g + row * P.D, row_bytes, bar0 + 8 * s);
            }
        }
    }

    // gain as packed bf16 pairs: in registers, except in the variant that is short of them (KEEP_T false), which parks
    // it in shared memory behind the ring and reads each vector back where it is used
    uint32_t gam[KEEP_T ? V : 1][4];
    const uint32_t gain_smem = ring + (uint32_t)stages * (uint32_t)P.stage_bytes;
    float2 acc[V][4];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int vi = tid + v * n;
        uint4 gw = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);   // ones
        if (GAIN && vi < nvec) gw = __ldg(reinterpret_cast<const uint4*>(P.gain) + vi);
        if (KEEP_T) {
            gam[v][0] = gw.x; gam[v][1] = gw.y; gam[v][2] = gw.z; gam[v][3] = gw.w;
        } else if (vi < nvec) {
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" :: "r"(gain_smem + (uint32_t)vi * 16u), "r"(gw.x), "r"(gw.y), "r"(gw.z), "r"(gw.w) : "memory");
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[v][j] = make_float2(0.0f, 0.0f);
    }
    __syncthreads();   // barriers initialised before anyone waits on them

    uint32_t it = 0;
    float r_next = P.rms[blockIdx.x];   // the row's RMS is fetched one iteration ahead (keeps the load off the critical path)
    for (int64_t row = blockIdx.x; row < P.T; row += stride, ++it) {
        const uint32_t s = it % (uint32_t)stages, parity = (it / (uint32_t)stages) & 1u;
        const uint32_t stage = ring + s * P.stage_bytes;
        const float r_row = r_next;
        if (row + stride < P.T) r_next = P.rms[row + stride];
        if (!mbar_wait_bounded(bar0 + 8 * s, parity)) abort_flag = 1;

        uint4 xw[V], gw[V];
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int vi = tid + v * n;
            if (vi < nvec) {
                xw[v] = lds_v4(stage + (uint32_t)vi * 16u);
                gw[v] = lds_v4(stage + half + (uint32_t)vi * 16u);
            } else {
                xw[v] = make_uint4(0, 0, 0, 0);
                gw[v] = make_uint4(0, 0, 0, 0);
            }
        }
        // a saved r of 0 marks a row of zeros (the forward emitted zeros for it): 1/r is taken as 0, so the row adds
        // nothing to dgamma and gets dX = 0 instead of 0 * inf = NaN
        const float inv_r = r_row == 0.0f ? 0.0f : __fdiv_rn(1.0f, r_row);

        // One pass over the thread's elements with  gi = g/r,  t = gi*gamma (= h/r):
        //   dgamma += x*gi ;  dot += t*x  (= sum_d h x / r) ;  later  dX = t - x * (dot/(D r^2)).
        // (two elements per instruction: packed binary32 multiply and fused multiply-add, each half an
        //  ordinary IEEE operation)
        float2 tt[KEEP_T ? V : 1][4];
        float2 dd = make_float2(0.f, 0.f);
        const float2 inv_r2 = make_float2(inv_r, inv_r);
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const uint32_t xa[4] = {xw[v].x, xw[v].y, xw[v].z, xw[v].w};
            const uint32_t ga[4] = {gw[v].x, gw[v].y, gw[v].z, gw[v].w};
            uint4 gq = make_uint4(0, 0, 0, 0);
            if (!KEEP_T && tid + v * n < nvec) gq = lds_v4(gain_smem + (uint32_t)(tid + v * n) * 16u);
            const uint32_t gm[4] = {KEEP_T ? gam[KEEP_T ? v : 0][0] : gq.x, KEEP_T ? gam[KEEP_T ? v : 0][1] : gq.y,
                                    KEEP_T ? gam[KEEP_T ? v : 0][2] : gq.z, KEEP_T ? gam[KEEP_T ? v : 0][3] : gq.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 x2 = bf16x2_to_f32x2(xa[j]);
                const float2 gi = mul2(bf16x2_to_f32x2(ga[j]), inv_r2);
                if (DGAIN) acc[v][j] = __ffma2_rn(x2, gi, acc[v][j]);
                const float2 t2 = GAIN ? mul2(gi, bf16x2_to_f32x2(gm[j])) : gi;
                if (KEEP_T) tt[v][j] = t2;
                dd = __ffma2_rn(t2, x2, dd);
            }
        }
        const float d0 = dd.x, d1 = dd.y;
        const float dot = warp_sum(d0 + d1);
        if (lane == 0) red[it & 1][warp] = dot;
        __syncthreads();   // row dot complete; every thread has read its part of the stage
        if (abort_flag) {
            // A wait ran out: the CTA requests no further copies and stops.  Copies already requested into the other
            // stages may still be in flight; one thread gives each of them a (shorter) bounded wait so that none lands
            // after this CTA's shared memory has been handed to another CTA, while the rest zero this CTA's row of
            // partial sums so that the column sum adds nothing stale.  dX rows from `row` on are left unwritten.
            if (DGAIN) {
                float* prow = P.partial + (int64_t)blockIdx.x * P.D;
                for (int i = tid; i < P.D; i += n) prow[i] = 0.0f;
            }
            if (tid == 0) {
                for (int j = 0; j < stages; ++j) {
                    const uint32_t itj = it + (uint32_t)j;
                    if (row + (int64_t)j * stride < P.T)
                        (void)mbar_wait_bounded(bar0 + 8 * (itj % (uint32_t)stages), (itj / (uint32_t)stages) & 1u, 1u << 16);
                }
                atomicAdd(&g_bwd_timeouts, 1u);
            }
            return;
        }
        if (tid == 0) {
            const int64_t next = row + (int64_t)stages * stride;
            if (next < P.T) {
                mbar_expect_tx(bar0 + 8 * s, 2 * row_bytes);
                bulk_load(stage, P.x + next * P.D, row_bytes, bar0 + 8 * s);
                bulk_load(stage + half, P.g + next * P.D, row_bytes, bar0 + 8 * s);
            }
        }
        float t = red[it & 1][0];
        for (int i = 1; i < nwarps; ++i) t += red[it & 1][i];
        const float c2 = t * invD * inv_r * inv_r;   // delta / r^3 with delta = (t * r) / D

#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int vi = tid + v * n;
            if (vi >= nvec) continue;
            const uint32_t xa[4] = {xw[v].x, xw[v].y, xw[v].z, xw[v].w};
            const uint32_t ga[4] = {gw[v].x, gw[v].y, gw[v].z, gw[v].w};
            uint4 gq = make_uint4(0, 0, 0, 0);
            if (!KEEP_T) gq = lds_v4(gain_smem + (uint32_t)vi * 16u);
            const uint32_t gm[4] = {KEEP_T ? gam[KEEP_T ? v : 0][0] : gq.x, KEEP_T ? gam[KEEP_T ? v : 0][1] : gq.y,
                                    KEEP_T ? gam[KEEP_T ? v : 0][2] : gq.z, KEEP_T ? gam[KEEP_T ? v : 0][3] : gq.w};
            float2 o[4];
            const float2 nc2 = make_float2(-c2, -c2);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float2 t2;
                if (KEEP_T) {
                    t2 = tt[v][j];
                } else {
                    const float2 gi = mul2(bf16x2_to_f32x2(ga[j]), inv_r2);
                    t2 = GAIN ? mul2(gi, bf16x2_to_f32x2(gm[j])) : gi;
                }
                o[j] = __ffma2_rn(bf16x2_to_f32x2(xa[j]), nc2, t2);
            }
            if (P.dx_is_fp32) {
                float* dp = static_cast<float*>(P.dx) + row * P.D + (int64_t)vi * 8;
                st_v4(dp, reinterpret_cast<const uint32_t*>(&o[0]));
                st_v4(dp + 4, reinterpret_cast<const uint32_t*>(&o[2]));
            } else {
                uint32_t pk[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) pk[j] = pack_bf16x2(o[j].x, o[j].y);
                st_v4(static_cast<uint16_t*>(P.dx) + row * P.D + (int64_t)vi * 8, pk);
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
                q[0] = make_float4(acc[v][0].x, acc[v][0].y, acc[v][1].x, acc[v][1].y);
                q[1] = make_float4(acc[v][2].x, acc[v][2].y, acc[v][3].x, acc[v][3].y);
            }
        }
    }
}

// dgain[j] = sum over the workspace rows, in a fixed order.  One CTA of 32 warps per C columns (D / C CTAs).  A warp
// load covers 32 / C rows x C columns; row slot q = warp * (32 / C) + lane / C adds rows q, q + Q, q + 2 Q, ... (Q = 1024 / C
// slots; ten loads in flight per thread), then the Q slot sums of a column are added in slot order.  C = 32 for wide
// rows (one 128-byte line per warp load), C = 8 for narrow ones, where D / 32 CTAs would leave most SMs idle while every
// CTA walks hundreds of partial rows.  Launched with programmatic stream serialisation so that its launch latency hides
// behind the tail of the main kernel; it waits for the main kernel's results before the first load.
constexpr int kReduceMaxRowsPerWarp = 10;   // loads a thread keeps in flight

template <int C>
__global__ void __launch_bounds__(1024) bwd_dgain_reduce_kernel(const float* __restrict__ partial, float* __restrict__ dgain,
                                                               int D, int parts)
{
    constexpr int Q = 1024 / C;                 // row slots per CTA
    __shared__ float s[Q][C + 1];
    const int c = threadIdx.x % C, q = threadIdx.x / C;
    const int col = blockIdx.x * C + c;
    pdl_prologue();
    float a = 0.0f;
    for (int base = q; base < parts; base += Q * kReduceMaxRowsPerWarp) {
        float v[kReduceMaxRowsPerWarp];
#pragma unroll
        for (int i = 0; i < kReduceMaxRowsPerWarp; ++i) {
            const int p = base + Q * i;
            v[i] = (col < D && p < parts) ? partial[(int64_t)p * D + col] : 0.0f;
        }
#pragma unroll
        for (int i = 0; i < kReduceMaxRowsPerWarp; ++i) a += v[i];
    }
    s[q][c] = a;
    __syncthreads();
    if (threadIdx.x < C && col < D) {
        float t = s[0][c];
#pragma unroll 8
        for (int i = 1; i < Q; ++i) t += s[i][c];
        dgain[col] = t;
    }
}

// threads per CTA, vectors per thread, ring stages and CTAs per SM for a row of D elements
struct BwdPlan { int threads, V, stages, stage_bytes, ctas_per_sm; size_t smem; };

// Threads per CTA, vectors per thread and CTAs per SM for rows of D elements.  Measured at 16384 rows:
//   D <= 2048: two vectors per thread in narrow CTAs and many of them (D = 2048: 128 threads x 5-6 CTAs per SM 36.1 / 29.5 us
//   with / without the gain gradient, against 45.4 / 38.1 us for 256 threads x 3; D = 1536: 96 x 6-8: 30.6 / 23.9 against
//   42.3 / 34.0; D = 1024: 64 x 8-12: 28.4 / 16.9 against 30.3 / 28.1 for 128 x 4).  The count follows the registers of the
//   variant (20 or 24 warps per SM); with the gain gradient at most 8 CTAs, because every CTA adds a row of partial sums.
//   D = 3072: 192 threads x 3 CTAs (49.7 / 44.3 us; 4 CTAs: 64.7 / 45.8).  D = 4096: 256 x 2 (65.2 / 59.2; 3 CTAs: 82.4 / 62.4).
//   Wider rows: 3 or 4 vectors per thread, 2 CTAs per SM; beyond 8192 elements 512 threads, 1 CTA.
static bool plan_bwd(int64_t D, bool dgain, BwdPlan* pl, bool gain = false, int64_t T = 0)
{
    if (D <= 0 || D % 8 != 0 || D > 16384) return false;
    const int64_t nvec = D / 8;
    int n, v, ctas;
    if (nvec <= 256) {
        v = nvec > 32 ? 2 : 1;
        n = (int)(((nvec + v - 1) / v + 31) / 32 * 32);
        const int warps = n / 32;
        ctas = dgain ? 20 / warps : 24 / warps;
        const int cap = dgain ? 8 : 12;
        ctas = ctas > cap ? cap : ctas;
    } else {
        n = MXN_BWD_THREADS;
        v = (int)((nvec + n - 1) / n);
        if (v > 4) {   // wide rows: up to 512 threads, three or four vectors per thread
            if (nvec > 4 * 512) return false;
            v = nvec > 3 * 512 ? 4 : 3;
        }
        // D = 8192 with the gain gradient: 512 threads x two vectors in one CTA per SM instead of 256 x four in two (the
        // four-vector variant with gain and gain gradient recomputes and parks the gain): 133.6 -> 127 us at 16384 rows,
        // 536 -> 480 us at 65536; narrower rows lose with it (D = 7168: 113 -> 121 us)
        // (taken without the gain gradient too, where it is level - 118.7 / 119.5 us - so that dX does not depend on
        // whether the gain gradient is asked for: the order of the row sum follows the thread layout)
        if (nvec > 960 && nvec <= 1024) v = 2;
        n = (int)(((nvec + v - 1) / v + 31) / 32 * 32);          // no more threads than v vectors each need (D = 3072: 192, not 256)
        ctas = n > MXN_BWD_THREADS ? 1 : (v == 2 && n <= 192) ? 3 : MXN_BWD_CTAS;
    }
    // Ring depth and CTAs per SM by row length and row count.  The defaults above were timed at 16384 rows; timing every
    // hidden size of the paper's grid at 16384, 32768 and 65536 rows with 2, 3 or the default number of stages and with fewer
    // CTAs per SM showed that long launches and long rows want fewer copies in flight (same DRAM bytes, measured; the DRAM
    // is busier: 82 % against 77 % of its cycles at [65536, 5120]).  What the rules below buy, default -> rule:
    //   rows wider than 8192 elements (512 threads): two stages, dX alone 4-10 % faster at 10240 ... 14336, level elsewhere;
    //   four vectors per thread in 256 threads (D = 7168, 8192) without the gain gradient: one CTA per SM, 3-13 % faster;
    //   three vectors per thread (D = 5120, 6144): two stages, with the gain gradient always (1-14 % faster), else from
    //     32768 rows on (5-7 %);
    //   D = 3072 (two vectors in 192 threads) from 32768 rows on: two stages, 2-10 % faster;
    //   D = 3584, 4096 (two vectors in 224 / 256 threads) with the gain gradient: three stages, 0-3 % faster;
    //   D <= 1792 with the gain gradient: three stages, 2-11 % faster;
    //   1536 <= D <= 2048 from 32768 rows on: a third fewer CTAs per SM with deeper rings, 3-20 % faster.
    // Over the 102 cells the geometric mean is 3 % faster, the worst cell 1.8 % slower (D = 10240, dX alone, 16384 rows).
    int forced_stages = 0;
    const bool many_rows = T >= 32768;
    if (n > MXN_BWD_THREADS && v >= 3) forced_stages = 2;
    else if (n > MXN_BWD_THREADS) forced_stages = 0;
    else if (v == 4 && !dgain) ctas = 1;
    else if (v == 3 && (dgain || many_rows)) forced_stages = 2;
    else if (v == 2 && n == 192 && nvec > 256 && many_rows) forced_stages = 2;
    else if (v == 2 && n > 192 && dgain) forced_stages = 3;
    else if (nvec <= 256) {
        if (dgain && D <= 1792) forced_stages = 3;
        else if (many_rows && D >= 1536) ctas = ctas >= 8 ? 5 : ctas >= 5 ? 4 : ctas;
        else if (!dgain && T >= 65536 && n == 64 && ctas > 8) ctas = 8;   // D = 1024, dX alone, 65536 rows: 69.0 -> 61.2 us
    }
    pl->threads = n;
    pl->V = v;                                                   // 1..4, each instantiated
    pl->ctas_per_sm = ctas;
    pl->stage_bytes = 2 * (int)((D * 2 + 127) / 128 * 128);     // x row + g row
    const int budget = 200 * 1024 / pl->ctas_per_sm;            // shared memory per CTA
    int st = budget / pl->stage_bytes;
    pl->stages = st < 2 ? 2 : (st > kBwdMaxStages ? kBwdMaxStages : st);
    if (forced_stages != 0 && forced_stages < pl->stages) pl->stages = forced_stages;
    pl->smem = (size_t)pl->stages * pl->stage_bytes;
    if (pl->V == 4 && gain && dgain) {   // room behind the ring for the gain of the variant that parks it there
        const size_t gain_bytes = (size_t)(D * 2 + 127) / 128 * 128;
        while (pl->stages > 2 && (pl->smem + gain_bytes) * pl->ctas_per_sm > 216 * 1024) pl->smem = (size_t)(--pl->stages) * pl->stage_bytes;
        pl->smem += gain_bytes;
    }
    return pl->smem <= 220 * 1024;
}

bool bwd_shape_supported(int64_t D)
{
    BwdPlan pl;
    return plan_bwd(D, true, &pl);
}

int bwd_parts(int64_t T, int64_t D)
{
    BwdPlan pl;
    // the plan with the gain gradient (the one that needs the workspace) for few rows: it has the most CTAs per SM, so
    // a workspace sized for T rows also serves every call with fewer rows
    if (!plan_bwd(D, true, &pl)) return 0;
    const int64_t cap = (int64_t)kSMs * pl.ctas_per_sm;
    return (int)(T < cap ? (T < 1 ? 1 : T) : cap);
}

typedef void (*bwd_fn)(const BwdParams);

template <int V, int NT>
static bwd_fn pick_bwd(bool gain, bool dgain)
{
    if (gain && dgain) return bwd_kernel<V, NT, true, true>;
    if (gain) return bwd_kernel<V, NT, true, false>;
    if (dgain) return bwd_kernel<V, NT, false, true>;
    return bwd_kernel<V, NT, false, false>;
}

cudaError_t launch_bwd(BwdParams P, cudaStream_t stream)
{
    const bool gain = P.gain != nullptr, dgain = P.dgain != nullptr;
    BwdPlan pl;
    if (!plan_bwd(P.D, dgain, &pl, gain, P.T)) return cudaErrorInvalidValue;
    P.stages = pl.stages;
    P.stage_bytes = pl.stage_bytes;
    {   // the grid of this variant (with the gain gradient it equals bwd_parts(T, D), which sized the workspace)
        const int64_t cap = (int64_t)kSMs * pl.ctas_per_sm;
        P.parts = (int)(P.T < cap ? P.T : cap);
    }
    // the kernel template below must be the one the plan sized shared memory for (the four-vector variant with gain and
    // gain gradient keeps the gain behind the ring): a mismatch is refused here instead of reaching the device
    if ((pl.threads > MXN_BWD_THREADS && (pl.V < 2 || pl.V > 4)) || pl.threads * pl.V < P.D / 8) return cudaErrorInvalidValue;
    bwd_fn fn;
    if (pl.threads > MXN_BWD_THREADS) fn = pl.V == 2 ? pick_bwd<2, 512>(gain, dgain) : pl.V == 3 ? pick_bwd<3, 512>(gain, dgain) : pick_bwd<4, 512>(gain, dgain);
    else if (pl.V == 1) fn = pick_bwd<1, MXN_BWD_THREADS>(gain, dgain);
    else if (pl.V == 2) fn = pl.threads <= 192 ? pick_bwd<2, 192>(gain, dgain) : pick_bwd<2, MXN_BWD_THREADS>(gain, dgain);   // 192: registers for 3+ CTAs per SM
    else if (pl.V == 3) fn = pick_bwd<3, MXN_BWD_THREADS>(gain, dgain);
    else fn = pick_bwd<4, MXN_BWD_THREADS>(gain, dgain);
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);
    if (e != cudaSuccess) return e;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)P.parts);
    cfg.blockDim = dim3((unsigned)pl.threads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, fn, P);
    if (e != cudaSuccess) return e;
    if (P.dgain != nullptr) {
        const bool narrow = P.D / 32 < 64;      // fewer than 64 CTAs of 32 columns: 8 columns per CTA instead (D = 1024: 29.2 -> 25.4 us)
        const int C = narrow ? 8 : 32;
        cfg.gridDim = dim3((unsigned)((P.D + C - 1) / C));
        cfg.blockDim = dim3(1024);
        cfg.dynamicSmemBytes = 0;
        const float* partial = P.partial;
        float* dgain = P.dgain;
        int D = P.D, parts = P.parts;
        e = narrow ? cudaLaunchKernelEx(&cfg, bwd_dgain_reduce_kernel<8>, partial, dgain, D, parts)
                   : cudaLaunchKernelEx(&cfg, bwd_dgain_reduce_kernel<32>, partial, dgain, D, parts);
    }
    return e;
}

// Host-only walk over every row length the backward accepts, with and without gain and gain gradient: counts the plans
// the launcher would refuse or whose shared memory would not fit the CTAs per SM they ask for.  No device is touched.
int64_t selftest_bwd_plans(int64_t max_D, int64_t* first_D, int* first_case)
{
    int64_t bad = 0;
    for (int64_t D = 8; D <= max_D; D += 8) {
        if (!bwd_shape_supported(D)) continue;
        for (int c = 0; c < 4; ++c) {
            const bool gain = (c & 2) != 0, dgain = (c & 1) != 0;
            bool ok = true;
            for (int big = 0; big < 2 && ok; ++big) {   // the plan depends on the number of rows
                const int64_t T = big ? (int64_t)1 << 20 : 1;
                BwdPlan pl;
                ok = plan_bwd(D, dgain, &pl, gain, T);
                if (ok) {
                    const size_t ring = (size_t)pl.stages * pl.stage_bytes;
                    const size_t parked = pl.V == 4 && gain && dgain ? (size_t)(D * 2 + 127) / 128 * 128 : 0;
                    BwdPlan ws;
                    ok = pl.V >= 1 && pl.V <= 4 && (pl.threads <= MXN_BWD_THREADS || (pl.threads <= 512 && pl.V >= 2))
                      && pl.threads % 32 == 0 && (int64_t)pl.threads * pl.V >= D / 8 && pl.stages >= 2 && pl.stages <= kBwdMaxStages
                      && pl.stage_bytes >= 4 * D && pl.smem == ring + parked
                      && pl.smem <= 227 * 1024                                             // one CTA's limit
                      && (pl.smem + 2048) * pl.ctas_per_sm <= 228 * 1024                   // the SM's, with static and reserved bytes
                      && pl.threads * pl.ctas_per_sm <= 2048
                      && plan_bwd(D, true, &ws) && (!dgain || pl.ctas_per_sm <= ws.ctas_per_sm);   // the workspace is sized by the few-rows plan
                }
            }
            if (!ok && bad++ == 0) {
                *first_D = D;
                *first_case = -(1 + c);
            }
        }
    }
    return bad;
}

cudaError_t read_timeouts(unsigned int* out)
{
    return cudaMemcpyFromSymbol(out, g_bwd_timeouts, sizeof(unsigned int));
}
cudaError_t reset_timeouts()
{
    const unsigned int zero = 0;
    return cudaMemcpyToSymbol(g_bwd_timeouts, &zero, sizeof(unsigned int));
}

// One warp waits, with the given number of polls, on an mbarrier that expects a transfer nobody issues: the wait
// must run out, be counted, and the kernel must return normally.
__global__ void __launch_bounds__(32) selftest_bounded_wait_kernel(uint32_t polls)
{
    __shared__ uint64_t bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x == 0 && !mbar_wait_bounded(b, 0, polls)) atomicAdd(&g_bwd_timeouts, 1u);
}
cudaError_t selftest_bounded_wait(unsigned int polls, cudaStream_t stream)
{
    selftest_bounded_wait_kernel<<<1, 32, 0, stream>>>(polls);
    return cudaGetLastError();
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
