// extern "C" entry points of libmxnorm: argument checks and dispatch only.
#include <mutex>

#include "../../include/mxnorm.h"
#include "mxn_internal.h"

namespace {

inline bool misaligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }

// the paper's printed correction constants RMS / G_p for Gaussian blocks (implementation appendix)
float paper_coef(int B, int p)
{
    switch (B * 4 + p) {
        case 16 * 4 + 1: return 0.4814f;
        case 16 * 4 + 2: return 0.4688f;
        case 32 * 4 + 1: return 0.4261f;
        case 32 * 4 + 2: return 0.4185f;
        case 64 * 4 + 1: return 0.3852f;
        case 64 * 4 + 2: return 0.3803f;
        default: return 0.0f;
    }
}

mxn_status check_common(const void* x, int64_t T, int64_t D, int B, const void* codes, const void* scales,
                        int round, int layout)
{
    if (T < 0 || D <= 0 || !mxn::fwd_shape_supported(D, B)) return MXN_ERR_SHAPE;
    if (round < 0 || round > MXN_ROUND_RCEIL_MAX) return MXN_ERR_ENUM;
    if (layout != MXN_SCALES_ROWMAJOR && layout != MXN_SCALES_SWIZZLE_128x4) return MXN_ERR_ENUM;
    if (T == 0) return MXN_OK;
    if (x == nullptr || codes == nullptr || scales == nullptr) return MXN_ERR_NULL;
    if (misaligned(x, 32) || misaligned(codes, 32)) return MXN_ERR_ALIGN;
    return MXN_OK;
}

// padding bytes of a tiled scale buffer are defined to be zero: clear the buffer when it has any
cudaError_t clear_scale_padding(void* scales, int64_t T, int64_t K, int layout, cudaStream_t s)
{
    if (layout == MXN_SCALES_SWIZZLE_128x4 && (T % 128 != 0 || K % 4 != 0))
        return cudaMemsetAsync(scales, 0, mxn_scale_bytes(T, K, MXN_SCALES_SWIZZLE_128x4), s);
    return cudaSuccess;
}

mxn_status run_fwd(int stat, bool nvfp4, const void* x, const void* gain, int64_t T, int64_t D, int B, int p,
                   float coef, float eps, float global_scale, void* codes, void* scales, float* rms,
                   int round, int layout, void* stream, int elem = mxn::ELEM_E4M3)
{
    mxn_status st = check_common(x, T, D, B, codes, scales, round, layout);
    if (st != MXN_OK || T == 0) return st;
    if (gain != nullptr && misaligned(gain, 16)) return MXN_ERR_ALIGN;
    if (rms != nullptr && misaligned(rms, 4)) return MXN_ERR_ALIGN;
    if (stat == mxn::STAT_MX) {
        if (p != 1 && p != 2) return MXN_ERR_SHAPE;
        if (coef == 0.0f) coef = paper_coef(B, p);
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    mxn::FwdParams P{};
    P.x = static_cast<const uint16_t*>(x);
    P.gain = static_cast<const uint16_t*>(gain);
    P.codes = static_cast<uint8_t*>(codes);
    P.scales = static_cast<uint8_t*>(scales);
    P.rms_out = rms;
    P.T = T;
    P.D = (int)D;
    P.K = (int)(D / B);
    P.p = p;
    P.coef = coef;
    P.eps = eps;
    P.global_scale = global_scale;
    P.round = round;
    P.layout = layout;
    P.elem = nvfp4 ? mxn::ELEM_E2M1 : elem;
    if (clear_scale_padding(scales, T, P.K, layout, s) != cudaSuccess) return MXN_ERR_CUDA;
    return mxn::launch_fwd(P, B, stat, nvfp4, s) == cudaSuccess ? MXN_OK : MXN_ERR_CUDA;
}

}  // namespace

extern "C" {

size_t mxn_scale_bytes(int64_t T, int64_t K, mxn_scale_layout layout)
{
    if (T < 0 || K < 0) return 0;
    if (layout == MXN_SCALES_ROWMAJOR) return (size_t)T * (size_t)K;
    if (layout == MXN_SCALES_SWIZZLE_128x4) return (size_t)((T + 127) / 128) * (size_t)((K + 3) / 4) * 512;
    return 0;
}

const char* mxn_status_string(mxn_status s)
{
    switch (s) {
        case MXN_OK: return "ok";
        case MXN_ERR_NULL: return "a required pointer is NULL";
        case MXN_ERR_SHAPE: return "unsupported shape, block size or p";
        case MXN_ERR_ALIGN: return "a pointer is not aligned as required";
        case MXN_ERR_ENUM: return "unknown rounding mode or scale layout";
        case MXN_ERR_WORKSPACE: return "workspace missing or too small";
        case MXN_ERR_CUDA: return "CUDA runtime error at launch";
        case MXN_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case MXN_ERR_TOO_LARGE: return "the problem needs more built-in scratch than the library holds";
        default: return "unknown status";
    }
}

mxn_status mxn_device_timeouts(unsigned int* count_out)
{
    unsigned int n = 0;
    if (cudaDeviceSynchronize() != cudaSuccess || mxn::read_timeouts(&n) != cudaSuccess) return MXN_ERR_CUDA;
    if (count_out != nullptr) *count_out = n;
    return n == 0 ? MXN_OK : MXN_ERR_TIMEOUT;
}

mxn_status mxn_device_timeouts_reset(void)
{
    return cudaDeviceSynchronize() == cudaSuccess && mxn::reset_timeouts() == cudaSuccess ? MXN_OK : MXN_ERR_CUDA;
}

mxn_status mxn_selftest_bounded_wait(unsigned int polls, void* cuda_stream)
{
    if (polls == 0 || polls > (1u << 16)) return MXN_ERR_SHAPE;
    return mxn::selftest_bounded_wait(polls, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? MXN_OK : MXN_ERR_CUDA;
}

mxn_status mxn_selftest_division(unsigned long long* mismatches_out)
{
    unsigned long long n = 0;
    if (mxn::selftest_division(&n) != cudaSuccess) return MXN_ERR_CUDA;
    if (mismatches_out != nullptr) *mismatches_out = n;
    return MXN_OK;
}

mxn_status mxn_selftest_dispatch(int64_t max_D, long long* missing_out, int64_t* first_D_out, int* first_case_out)
{
    if (missing_out == nullptr) return MXN_ERR_NULL;
    if (max_D < 16) return MXN_ERR_SHAPE;
    int64_t first_D = 0;
    int first_case = 0;
    int64_t missing = mxn::selftest_dispatch(max_D, &first_D, &first_case);
    {
        int64_t d = 0;
        int c = 0;
        const int64_t bad = mxn::selftest_bwd_plans(max_D, &d, &c);
        if (missing == 0 && bad != 0) {
            first_D = d;
            first_case = c;
        }
        missing += bad;
    }
    *missing_out = (long long)missing;
    if (first_D_out != nullptr) *first_D_out = first_D;
    if (first_case_out != nullptr) *first_case_out = first_case;
    return MXN_OK;
}

mxn_status mx_cast(const void* x_bf16, int64_t T, int64_t D, int block, void* codes_u8, void* scales_u8,
                   mxn_round round, mxn_scale_layout layout, void* cuda_stream)
{
    return run_fwd(mxn::STAT_NONE, false, x_bf16, nullptr, T, D, block, 2, 1.0f, 0.0f, 1.0f, codes_u8, scales_u8,
                   nullptr, round, layout, cuda_stream);
}

mxn_status rmsnorm_mxfp8_fwd(const void* x_bf16, const void* gain_bf16_or_null, int64_t T, int64_t D, int block,
                             float eps, void* codes_u8, void* scales_u8, float* rms_out_or_null,
                             mxn_round round, mxn_scale_layout layout, void* cuda_stream)
{
    return run_fwd(mxn::STAT_RMS, false, x_bf16, gain_bf16_or_null, T, D, block, 2, 1.0f, eps, 1.0f, codes_u8,
                   scales_u8, rms_out_or_null, round, layout, cuda_stream);
}

mxn_status mxnorm_fwd(const void* x_bf16, const void* gain_bf16_or_null, int64_t T, int64_t D, int block, int p,
                      float coef_or_0, float eps, void* codes_u8, void* scales_u8, float* rms_est_out_or_null,
                      mxn_round round, mxn_scale_layout layout, void* cuda_stream)
{
    return run_fwd(mxn::STAT_MX, false, x_bf16, gain_bf16_or_null, T, D, block, p, coef_or_0, eps, 1.0f, codes_u8,
                   scales_u8, rms_est_out_or_null, round, layout, cuda_stream);
}

mxn_status mxnorm_nvfp4_fwd(const void* x_bf16, int64_t T, int64_t D, int p, float coef_or_0, float eps,
                            float global_scale, void* codes_u8_packed, void* scales_e4m3,
                            float* rms_est_out_or_null, mxn_scale_layout layout, void* cuda_stream)
{
    return run_fwd(mxn::STAT_MX, true, x_bf16, nullptr, T, D, 16, p, coef_or_0, eps, global_scale, codes_u8_packed,
                   scales_e4m3, rms_est_out_or_null, MXN_ROUND_RCEIL_POW2, layout, cuda_stream);
}

mxn_status mx_cast_nvfp4(const void* x_bf16, int64_t T, int64_t D, float global_scale, void* codes_u8_packed,
                      void* scales_e4m3, mxn_scale_layout layout, void* cuda_stream)
{
    return run_fwd(mxn::STAT_NONE, true, x_bf16, nullptr, T, D, 16, 2, 1.0f, 0.0f, global_scale, codes_u8_packed,
                   scales_e4m3, nullptr, MXN_ROUND_RCEIL_POW2, layout, cuda_stream);
}

mxn_status rmsnorm_nvfp4_fwd(const void* x_bf16, int64_t T, int64_t D, float eps, float global_scale,
                             void* codes_u8_packed, void* scales_e4m3, float* rms_out_or_null,
                             mxn_scale_layout layout, void* cuda_stream)
{
    return run_fwd(mxn::STAT_RMS, true, x_bf16, nullptr, T, D, 16, 2, 1.0f, eps, global_scale, codes_u8_packed,
                   scales_e4m3, rms_out_or_null, MXN_ROUND_RCEIL_POW2, layout, cuda_stream);
}

mxn_status mxnorm_add_fwd(const void* x_bf16, const void* residual_bf16, int64_t T, int64_t D, int block, int p,
                          float coef_or_0, float eps, void* h_out_bf16, void* codes_u8, void* scales_u8,
                          float* rms_est_out_or_null, mxn_scale_layout layout, void* cuda_stream)
{
    mxn_status st = check_common(x_bf16, T, D, block, codes_u8, scales_u8, MXN_ROUND_RCEIL_POW2, layout);
    if (st != MXN_OK || T == 0) return st;
    if (residual_bf16 == nullptr || h_out_bf16 == nullptr) return MXN_ERR_NULL;
    if (misaligned(residual_bf16, 32) || misaligned(h_out_bf16, 32)) return MXN_ERR_ALIGN;
    if (p != 1 && p != 2) return MXN_ERR_SHAPE;
    if (rms_est_out_or_null != nullptr && misaligned(rms_est_out_or_null, 4)) return MXN_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    mxn::FwdParams P{};
    P.x = static_cast<const uint16_t*>(x_bf16);
    P.residual = static_cast<const uint16_t*>(residual_bf16);
    P.h_out = static_cast<uint16_t*>(h_out_bf16);
    P.codes = static_cast<uint8_t*>(codes_u8);
    P.scales = static_cast<uint8_t*>(scales_u8);
    P.rms_out = rms_est_out_or_null;
    P.T = T;
    P.D = (int)D;
    P.K = (int)(D / block);
    P.p = p;
    P.coef = coef_or_0 == 0.0f ? paper_coef(block, p) : coef_or_0;
    P.eps = eps;
    P.global_scale = 1.0f;
    P.round = MXN_ROUND_RCEIL_POW2;
    P.layout = layout;
    P.elem = mxn::ELEM_E4M3;
    if (clear_scale_padding(scales_u8, T, P.K, layout, s) != cudaSuccess) return MXN_ERR_CUDA;
    return mxn::launch_fwd(P, block, mxn::STAT_MX, false, s) == cudaSuccess ? MXN_OK : MXN_ERR_CUDA;
}

mxn_status mxnorm_postround_fwd(const void* x_bf16, int64_t T, int64_t D, int block, float eps, void* codes_u8,
                                void* scales_u8, float* rms_est_out_or_null, mxn_scale_layout layout, void* cuda_stream)
{
    mxn_status st = check_common(x_bf16, T, D, block, codes_u8, scales_u8, MXN_ROUND_RCEIL_POW2, layout);
    if (st != MXN_OK || T == 0) return st;
    if (mxn::postround_prepare(block) != cudaSuccess) return MXN_ERR_CUDA;
    return run_fwd(mxn::STAT_POSTROUND, false, x_bf16, nullptr, T, D, block, 2, 1.0f, eps, 1.0f, codes_u8, scales_u8,
                   rms_est_out_or_null, MXN_ROUND_RCEIL_POW2, layout, cuda_stream);
}

mxn_status mx_cast_fp4(const void* x_bf16, int64_t T, int64_t D, int block, void* codes_u8_packed, void* scales_u8,
                       mxn_scale_layout layout, void* cuda_stream)
{
    return run_fwd(mxn::STAT_NONE, false, x_bf16, nullptr, T, D, block, 2, 1.0f, 0.0f, 1.0f, codes_u8_packed, scales_u8,
                   nullptr, MXN_ROUND_RCEIL_POW2, layout, cuda_stream, mxn::ELEM_E2M1);
}

mxn_status rmsnorm_mxfp4_fwd(const void* x_bf16, int64_t T, int64_t D, int block, float eps, void* codes_u8_packed,
                             void* scales_u8, float* rms_out_or_null, mxn_scale_layout layout, void* cuda_stream)
{
    return run_fwd(mxn::STAT_RMS, false, x_bf16, nullptr, T, D, block, 2, 1.0f, eps, 1.0f, codes_u8_packed, scales_u8,
                   rms_out_or_null, MXN_ROUND_RCEIL_POW2, layout, cuda_stream, mxn::ELEM_E2M1);
}

mxn_status mxnorm_mxfp4_fwd(const void* x_bf16, int64_t T, int64_t D, int block, int p, float coef_or_0, float eps,
                            void* codes_u8_packed, void* scales_u8, float* rms_est_out_or_null,
                            mxn_scale_layout layout, void* cuda_stream)
{
    return run_fwd(mxn::STAT_MX, false, x_bf16, nullptr, T, D, block, p, coef_or_0, eps, 1.0f, codes_u8_packed, scales_u8,
                   rms_est_out_or_null, MXN_ROUND_RCEIL_POW2, layout, cuda_stream, mxn::ELEM_E2M1);
}

namespace {
mxn_status run_transposed(const void* x_bf16, const float* rms_or_null, int64_t T, int64_t D, float eps, void* codes_t_u8,
                          void* scales_t_u8, int round, int layout, int elem, void* cuda_stream);
}

mxn_status mx_cast_e5m2(const void* x_bf16, int64_t T, int64_t D, int block, void* codes_u8, void* scales_u8,
                        mxn_scale_layout layout, void* cuda_stream)
{
    return run_fwd(mxn::STAT_NONE, false, x_bf16, nullptr, T, D, block, 2, 1.0f, 0.0f, 1.0f, codes_u8, scales_u8, nullptr,
                   MXN_ROUND_RCEIL_POW2, layout, cuda_stream, mxn::ELEM_E5M2);
}

mxn_status mx_cast_transposed_e5m2(const void* x_bf16, int64_t T, int64_t D, void* codes_t_u8, void* scales_t_u8,
                                   mxn_scale_layout layout, void* cuda_stream)
{
    return run_transposed(x_bf16, nullptr, T, D, 0.0f, codes_t_u8, scales_t_u8, MXN_ROUND_RCEIL_POW2, layout, mxn::ELEM_E5M2,
                          cuda_stream);
}

mxn_status mx_cast_transposed(const void* x_bf16, const float* rms_or_null, int64_t T, int64_t D, float eps,
                              void* codes_t_u8, void* scales_t_u8, mxn_round round, mxn_scale_layout layout,
                              void* cuda_stream)
{
    return run_transposed(x_bf16, rms_or_null, T, D, eps, codes_t_u8, scales_t_u8, round, layout, mxn::ELEM_E4M3, cuda_stream);
}

namespace {
mxn_status run_transposed(const void* x_bf16, const float* rms_or_null, int64_t T, int64_t D, float eps, void* codes_t_u8,
                          void* scales_t_u8, int round, int layout, int elem, void* cuda_stream)
{
    if (T < 0 || D <= 0 || T % 32 != 0 || D % 4 != 0 || D > 0x7FFFFFFF || T / 128 > 65535) return MXN_ERR_SHAPE;
    if (round < 0 || round > MXN_ROUND_RCEIL_MAX) return MXN_ERR_ENUM;
    if (layout != MXN_SCALES_ROWMAJOR && layout != MXN_SCALES_SWIZZLE_128x4) return MXN_ERR_ENUM;
    if (T == 0) return MXN_OK;
    if (x_bf16 == nullptr || codes_t_u8 == nullptr || scales_t_u8 == nullptr) return MXN_ERR_NULL;
    if (misaligned(x_bf16, 8) || misaligned(codes_t_u8, 32) || (rms_or_null != nullptr && misaligned(rms_or_null, 4)))
        return MXN_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (clear_scale_padding(scales_t_u8, D, T / 32, layout, s) != cudaSuccess) return MXN_ERR_CUDA;
    mxn::TransposedParams P{};
    P.x = static_cast<const uint16_t*>(x_bf16);
    P.rms = rms_or_null;
    P.codes = static_cast<uint8_t*>(codes_t_u8);
    P.scales = static_cast<uint8_t*>(scales_t_u8);
    P.T = T;
    P.D = (int)D;
    P.eps = eps;
    P.round = round;
    P.layout = layout;
    P.elem = elem;
    return mxn::launch_cast_transposed(P, s) == cudaSuccess ? MXN_OK : MXN_ERR_CUDA;
}
}  // namespace

mxn_status mxnorm_bwd(const void* x_bf16, const void* grad_out_bf16, const void* gain_bf16_or_null,
                      const float* rms, int64_t T, int64_t D, void* dx, int dx_is_fp32, float* dgain_f32_or_null,
                      void* workspace, size_t workspace_bytes, void* cuda_stream)
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
    if (misaligned(x_bf16, 16) || misaligned(grad_out_bf16, 16) || misaligned(dx, 16) || misaligned(rms, 4) ||
        (gain_bf16_or_null != nullptr && misaligned(gain_bf16_or_null, 16)) ||
        (dgain_f32_or_null != nullptr && misaligned(dgain_f32_or_null, 16)))
        return MXN_ERR_ALIGN;
    if (dgain_f32_or_null != nullptr) {
        if (workspace == nullptr || workspace_bytes < mxnorm_bwd_workspace_bytes(T, D)) return MXN_ERR_WORKSPACE;
        if (misaligned(workspace, 16)) return MXN_ERR_ALIGN;
    }
    mxn::BwdParams P{};
    P.x = static_cast<const uint16_t*>(x_bf16);
    P.g = static_cast<const uint16_t*>(grad_out_bf16);
    P.gain = static_cast<const uint16_t*>(gain_bf16_or_null);
    P.rms = rms;
    P.dx = dx;
    P.dgain = dgain_f32_or_null;
    P.partial = static_cast<float*>(workspace);
    P.T = T;
    P.D = (int)D;
    P.dx_is_fp32 = dx_is_fp32 != 0;
    P.parts = mxn::bwd_parts(T, D);
    return mxn::launch_bwd(P, s) == cudaSuccess ? MXN_OK : MXN_ERR_CUDA;
}

size_t mxnorm_bwd_workspace_bytes(int64_t T, int64_t D)
{
    if (T <= 0 || D <= 0 || !mxn::bwd_shape_supported(D)) return 0;
    return (size_t)mxn::bwd_parts(T, D) * (size_t)D * sizeof(float);
}

// ---- host-memory front end ----------------------------------------------------------------------
namespace {

struct HostPipe {
    bool ready = false;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t fork = nullptr, copied = nullptr, join = nullptr;
};
constexpr int kMaxDevices = 64;
HostPipe g_pipes[kMaxDevices];
std::mutex g_pipes_mutex;

// call with g_pipes_mutex held
HostPipe* host_pipe()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    HostPipe& hp = g_pipes[dev];
    if (!hp.ready) {
        if (cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&hp.fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&hp.copied, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&hp.join, cudaEventDisableTiming) != cudaSuccess)
            return nullptr;
        hp.ready = true;
    }
    return &hp;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
constexpr int64_t kHostChunkRows = 2048;   // multiple of the 128-row scale tile

}  // namespace

size_t mxnorm_fwd_host_workspace_bytes(int64_t T, int64_t D, int block, mxn_scale_layout layout)
{
    if (T <= 0 || D <= 0 || !mxn::fwd_shape_supported(D, block)) return 0;
    const size_t sb = mxn_scale_bytes(T, D / block, layout);
    if (sb == 0) return 0;
    return align_up((size_t)T * D * 2, 256) + align_up((size_t)T * D, 256) + align_up(sb, 256) +
           align_up((size_t)T * 4, 256);
}

mxn_status mxnorm_fwd_host(const void* x_host_bf16, int64_t T, int64_t D, int block, int p, float coef_or_0,
                           float eps, void* codes_host, void* scales_host, float* rms_est_host_or_null,
                           mxn_round round, mxn_scale_layout layout, void* workspace, size_t workspace_bytes,
                           void* cuda_stream)
{
    if (T < 0 || D <= 0 || !mxn::fwd_shape_supported(D, block) || (p != 1 && p != 2)) return MXN_ERR_SHAPE;
    if (round < 0 || round > MXN_ROUND_RCEIL_MAX) return MXN_ERR_ENUM;
    if (layout != MXN_SCALES_ROWMAJOR && layout != MXN_SCALES_SWIZZLE_128x4) return MXN_ERR_ENUM;
    if (T == 0) return MXN_OK;
    if (x_host_bf16 == nullptr || codes_host == nullptr || scales_host == nullptr) return MXN_ERR_NULL;
    if (workspace == nullptr || workspace_bytes < mxnorm_fwd_host_workspace_bytes(T, D, block, layout))
        return MXN_ERR_WORKSPACE;
    if (misaligned(workspace, 256)) return MXN_ERR_ALIGN;
    // the internal streams and events of a device are shared by every call on it: one call enqueues at a time
    std::lock_guard<std::mutex> pipe_lock(g_pipes_mutex);
    HostPipe* hp = host_pipe();
    if (hp == nullptr) return MXN_ERR_CUDA;
    cudaStream_t user = static_cast<cudaStream_t>(cuda_stream);

    const int64_t K = D / block;
    const size_t sbytes = mxn_scale_bytes(T, K, layout);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    uint16_t* dx = reinterpret_cast<uint16_t*>(base);
    uint8_t* dcodes = base + align_up((size_t)T * D * 2, 256);
    uint8_t* dscales = dcodes + align_up((size_t)T * D, 256);
    float* drms = reinterpret_cast<float*>(dscales + align_up(sbytes, 256));
    const uint16_t* hx = static_cast<const uint16_t*>(x_host_bf16);
    uint8_t* hcodes = static_cast<uint8_t*>(codes_host);
    uint8_t* hscales = static_cast<uint8_t*>(scales_host);

    if (cudaEventRecord(hp->fork, user) != cudaSuccess) return MXN_ERR_CUDA;   // nothing forked yet
    bool ok = cudaStreamWaitEvent(hp->in, hp->fork, 0) == cudaSuccess &&
              cudaStreamWaitEvent(hp->out, hp->fork, 0) == cudaSuccess;
    mxn_status failed = MXN_OK;
    const bool tiled = layout == MXN_SCALES_SWIZZLE_128x4;
    const int64_t tiles_per_row = (K + 3) / 4;
    for (int64_t r0 = 0; ok && r0 < T; r0 += kHostChunkRows) {
        const int64_t rows = (T - r0 < kHostChunkRows) ? T - r0 : kHostChunkRows;
        ok = cudaMemcpyAsync(dx + r0 * D, hx + r0 * D, (size_t)rows * D * 2, cudaMemcpyHostToDevice, hp->in) == cudaSuccess &&
             cudaEventRecord(hp->copied, hp->in) == cudaSuccess &&
             cudaStreamWaitEvent(hp->out, hp->copied, 0) == cudaSuccess;
        if (!ok) break;
        // a chunk starts on a 128-row boundary, so its scales are a contiguous slice in either layout
        const size_t soff = tiled ? (size_t)(r0 / 128) * tiles_per_row * 512 : (size_t)r0 * K;
        const size_t slen = tiled ? (size_t)((rows + 127) / 128) * tiles_per_row * 512 : (size_t)rows * K;
        mxn_status st = run_fwd(mxn::STAT_MX, false, dx + r0 * D, nullptr, rows, D, block, p, coef_or_0, eps, 1.0f,
                                dcodes + r0 * D, dscales + soff, drms + r0, round, layout, hp->out);
        if (st != MXN_OK) {   // leave through the join below: the chunks already enqueued must stay ordered
            failed = st;
            break;
        }
        ok = cudaMemcpyAsync(hcodes + r0 * D, dcodes + r0 * D, (size_t)rows * D, cudaMemcpyDeviceToHost, hp->out) == cudaSuccess &&
             cudaMemcpyAsync(hscales + soff, dscales + soff, slen, cudaMemcpyDeviceToHost, hp->out) == cudaSuccess;
        if (ok && rms_est_host_or_null != nullptr)
            ok = cudaMemcpyAsync(rms_est_host_or_null + r0, drms + r0, (size_t)rows * 4, cudaMemcpyDeviceToHost, hp->out) == cudaSuccess;
    }
    // Join on every path that forked: the caller's stream waits for both internal streams, so whatever was enqueued
    // (copies into the caller's buffers included) is ordered before anything the caller enqueues next.
    const bool joined = cudaEventRecord(hp->copied, hp->in) == cudaSuccess &&
                        cudaStreamWaitEvent(hp->out, hp->copied, 0) == cudaSuccess &&
                        cudaEventRecord(hp->join, hp->out) == cudaSuccess &&
                        cudaStreamWaitEvent(user, hp->join, 0) == cudaSuccess;
    if (failed != MXN_OK) return failed;
    return ok && joined ? MXN_OK : MXN_ERR_CUDA;
}

}  // extern "C"
