// Host-side declarations shared by the libmxnorm translation units (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace mxn {

enum { STAT_NONE = 0, STAT_RMS = 1, STAT_MX = 2, STAT_POSTROUND = 3 };
enum { ELEM_E4M3 = 0, ELEM_E2M1 = 1, ELEM_E5M2 = 2 };

struct FwdParams {
    const uint16_t* x;      // bf16 [T, D]
    const uint16_t* gain;   // bf16 [D] or nullptr
    const uint16_t* residual; // bf16 [T, D] or nullptr: added to x before the norm (fused residual add)
    uint16_t* h_out;        // bf16 [T, D]: x + residual, written when residual is given
    uint8_t* codes;         // [T, D] (E4M3) or [T, D/2] (E2M1 pairs)
    uint8_t* scales;        // row-major [T, K] or 128x4-tiled
    float* rms_out;         // [T] or nullptr
    int64_t T;
    int D, K;
    int p;
    float coef, eps, global_scale;
    int round, layout;
    int elem;               // ELEM_E4M3 (one byte per element) or ELEM_E2M1 (two elements per byte)
    // filled by the launcher
    int wpr, npass, rows_per_cta, tiles_per_row;
    int chunks;             // per-lane pieces of a row: K * (lanes per block)
    int pr_table;           // post-round estimator: index of the block size's f^-1 table
    double inv_count;       // 1/K (MXNorm) or 1/D (RMSNorm) when that is a power of two (exact), else 0
};

bool fwd_shape_supported(int64_t D, int B);
cudaError_t launch_fwd(FwdParams P, int B, int stat, bool nvfp4, cudaStream_t stream);
cudaError_t selftest_division(unsigned long long* mismatches_host);
int64_t selftest_dispatch(int64_t max_D, int64_t* first_D, int* first_case);   // host only
int64_t selftest_bwd_plans(int64_t max_D, int64_t* first_D, int* first_case);  // host only
cudaError_t postround_prepare(int B);   // uploads the f^-1 table for block size B to the current device (once)

struct TransposedParams {
    const uint16_t* x;      // bf16 [T, D]
    const float* rms;       // [T] or nullptr (rho = 1)
    uint8_t* codes;         // [D, T]
    uint8_t* scales;        // [D, T/32] row-major or 128x4-tiled (rows = D)
    int64_t T;
    int D;
    float eps;
    int round, layout;
    int elem;               // ELEM_E4M3 or ELEM_E5M2
    int KT, tiles_per_row;  // filled by the launcher
};
cudaError_t launch_cast_transposed(TransposedParams P, cudaStream_t stream);

struct BwdParams {
    const uint16_t* x;      // bf16 [T, D]
    const uint16_t* g;      // bf16 [T, D]
    const uint16_t* gain;   // bf16 [D] or nullptr
    const float* rms;       // [T]
    void* dx;               // bf16 or fp32 [T, D]
    float* dgain;           // [D] or nullptr
    float* partial;         // workspace [P, D] fp32
    int64_t T;
    int D;
    int dx_is_fp32;
    int parts;              // number of partial rows in the workspace (= CTAs of the main kernel)
    int stages, stage_bytes; // shared-memory ring (filled by the launcher)
};

bool bwd_shape_supported(int64_t D);
int bwd_parts(int64_t T, int64_t D);
cudaError_t launch_bwd(BwdParams P, cudaStream_t stream);
// bounded device-side waits that ran out (the backward's bulk-copy ring is the only code that waits)
cudaError_t read_timeouts(unsigned int* out);
cudaError_t reset_timeouts();
cudaError_t selftest_bounded_wait(unsigned int polls, cudaStream_t stream);

}  // namespace mxn
