/*
 * libmxnorm - C ABI of the B200 (sm_100a) MXNorm hot path.
 *
 * MXNorm (Algorithm 2 of the paper) replaces "RMSNorm followed by an MXFP8 cast"
 * (Algorithm 1) by one pass that takes every block's absmax, estimates the row RMS
 * from those K = D/B block statistics and emits the normalised tensor directly as
 * block-scaled low-precision codes.
 *
 * Conventions shared by every entry point unless stated otherwise
 * ----------------------------------------------------------------
 *  - Tensor pointers are DEVICE pointers owned by the caller.  The library never
 *    allocates, frees or synchronises; work is enqueued on `cuda_stream` (a
 *    cudaStream_t passed as void*, NULL = the legacy default stream) of the
 *    device that is current when the call is made.
 *  - X is bf16 [T, D], row-major, contiguous, base address 32-byte aligned (read with 32-byte loads).
 *    T >= 0 rows (tokens), D hidden size, `block` = B, K = D / B blocks per row.
 *    Supported: B in {16, 32, 64} (NVFP4: B = 16 fixed), D % B == 0,
 *    D <= 32768 (backward: D % 8 == 0, D <= 16384).  T == 0 returns MXN_OK without a launch.
 *  - codes: one byte per element (E4M3, OCP "fn": bias 7, max 448, no infinity),
 *    [T, D] row-major; written with 32-byte stores: base 32-byte aligned.
 *  - scales: one byte per block.  MXN_SCALES_ROWMAJOR: [T, K].
 *    MXN_SCALES_SWIZZLE_128x4: the tiled layout block-scaled tensor-core GEMMs
 *    read - rows padded to a multiple of 128, scale columns to a multiple of 4,
 *    each (128 rows x 4 scales) tile 512 contiguous bytes, tiles row-tile major;
 *    byte offset of (r, c) =
 *      ((r/128) * ceil(K/4) + c/4) * 512 + (r%32) * 16 + ((r%128)/32) * 4 + c%4.
 *    The buffer must hold mxn_scale_bytes(T, K, layout) bytes; padding bytes are
 *    written as 0.
 *  - Launch semantics: kernels are launched with programmatic stream serialisation.  Each kernel
 *    waits, before it reads or writes any value, until the preceding kernel of the stream has completed
 *    and its writes are visible, so ordering and results are those of ordinary stream order; what
 *    overlaps the tail of the previous kernel is the launch latency and L2 prefetch hints for the first
 *    input rows (a prefetch consumes no value; L2 is the point of coherence, so a line requested early
 *    and then written by the previous kernel is read with its new contents).  A kernel that FOLLOWS a
 *    libmxnorm kernel and is itself launched with the programmatic attribute must do the same wait
 *    (griddepcontrol.wait / cudaGridDependencySynchronize) before reading libmxnorm's outputs;
 *    ordinary launches need nothing.
 *  - Stream capture: every device-pointer entry point only enqueues kernels (and, for a tiled scale
 *    buffer with padding, one memset) on `cuda_stream`, so it may be called while that stream is being
 *    captured into a CUDA graph; the exceptions are stated at the entry points concerned (the first
 *    call of mxnorm_postround_fwd per block size and the first call of mxnorm_bwd_noalloc and of
 *    mxnorm_fwd_host per device do one-time set-up that is not capturable).
 *  - Outputs are fully overwritten.  Inputs must be finite; results for NaN/Inf
 *    inputs are unspecified (no fault).
 *  - Every function returns a status; nothing aborts, throws or prints.  Argument
 *    errors are detected before anything is enqueued.  CUDA launch failures map
 *    to MXN_ERR_CUDA.
 *  - Arithmetic contract (what the CPU oracle states and the tests compare):
 *    block absmaxes exact; row statistic accumulated in binary64 and rounded once
 *    to binary32; every element-wise product one IEEE binary32 operation; E8M0
 *    scales by exact exponent tests; element codes round-to-nearest-even,
 *    saturating.  Normalisation factors 1/(r + eps) are 0 for a zero denominator (a row of zeros
 *    stays zero) and saturate at the largest finite binary32 instead of overflowing.
 */
#ifndef MXNORM_H_
#define MXNORM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MXN_OK = 0,
    MXN_ERR_NULL = 1,      /* a required pointer is NULL */
    MXN_ERR_SHAPE = 2,     /* T < 0, D <= 0, D % B != 0, unsupported B or D, bad p */
    MXN_ERR_ALIGN = 3,     /* a pointer misses the alignment stated above */
    MXN_ERR_ENUM = 4,      /* unknown rounding mode / layout */
    MXN_ERR_WORKSPACE = 5, /* workspace NULL or smaller than the query says */
    MXN_ERR_CUDA = 6,      /* the CUDA runtime reported an error at launch */
    MXN_ERR_TIMEOUT = 7,   /* a bounded device-side wait ran out (reported by mxn_device_timeouts) */
    MXN_ERR_TOO_LARGE = 8  /* the problem needs more built-in scratch than the library holds */
} mxn_status;

/* Power-of-two rounding of the block scale (Section 3.2: "implementation-defined").
 *   RCEIL_POW2 : the paper's rule - round UP the quotient absmax / 2^emax, where 2^emax
 *                is the largest power of two of the element format (256 for E4M3):
 *                S = 2^(ceil(log2 absmax) - emax).  Codes never exceed 2^emax.
 *   FLOOR_OCP  : S = 2^(floor(log2 absmax) - emax) (OCP MX specification); codes saturate.
 *   RCEIL_MAX  : S = 2^ceil(log2(absmax / max_elem)) with max_elem = 448 (one binary32
 *                division). */
typedef enum { MXN_ROUND_RCEIL_POW2 = 0, MXN_ROUND_FLOOR_OCP = 1, MXN_ROUND_RCEIL_MAX = 2 } mxn_round;

typedef enum { MXN_SCALES_ROWMAJOR = 0, MXN_SCALES_SWIZZLE_128x4 = 1 } mxn_scale_layout;

/* Bytes a scale buffer needs for T rows of K scales in the given layout
 * (T*K row-major; ceil(T/128)*ceil(K/4)*512 tiled).  Returns 0 for a bad layout. */
size_t mxn_scale_bytes(int64_t T, int64_t K, mxn_scale_layout layout);

const char* mxn_status_string(mxn_status s);

/* Diagnostics: the one kernel that waits on asynchronous copies (the backward, which feeds its rows through a ring of
 * shared-memory stages filled by the bulk-copy engine) bounds every wait.  A wait that runs out makes its thread block
 * stop and bumps a device-side counter instead of hanging: the block requests no further copies, gives the copies it
 * had already requested a second, shorter bounded wait, writes zeros for its share of the dgain partial sums and
 * returns.  After such an event the dx rows that block had not reached yet are unwritten and dgain lacks that block's
 * rows: the outputs of the affected launch are incomplete and must be discarded.
 *   mxn_device_timeouts synchronises the device, stores the number of such events since the library was loaded (or
 *   since the last reset) into *count_out and returns MXN_ERR_TIMEOUT when it is non-zero, else MXN_OK.
 *   mxn_device_timeouts_reset synchronises the device and sets the counter back to 0.
 *   mxn_selftest_bounded_wait (a test utility) enqueues one warp that waits `polls` times (1..65536) on a barrier
 *   nobody completes: the wait must run out, be counted exactly once, and the kernel must return normally. */
mxn_status mxn_device_timeouts(unsigned int* count_out);
mxn_status mxn_device_timeouts_reset(void);
mxn_status mxn_selftest_bounded_wait(unsigned int polls, void* cuda_stream);

/* Diagnostics: the NVFP4 kernels replace the IEEE divisions by 6 and by an E4M3 scale with a multiply and two
 * fused multiply-adds that give the same correctly rounded quotient.  This call re-checks that claim on the
 * current device for every binary32 numerator between 2^-100 and 2^100 and every divisor the kernels use
 * (about a second; it allocates and frees 8 bytes of device memory and synchronises the device - a test
 * utility, not part of the hot path).  *mismatches_out receives the number of differing quotients (0). */
mxn_status mxn_selftest_division(unsigned long long* mismatches_out);

/* Diagnostics, host only (no device is touched): walks every row length D <= max_D that the forward entry points
 * accept, for each block size, row statistic, element format, gain / residual option and scale rounding rule they can
 * ask for, and counts the combinations for which the launcher would find no compiled kernel (expected: 0, i.e. a shape
 * that passes the argument checks can always be launched).  *missing_out receives the count; when it is non-zero
 * *first_D_out / *first_case_out (either may be NULL) receive the first such row length and a decimal code
 * ((block * 10 + variant) * 10 + statistic) * 10 + rounding rule, with variant 0 E4M3, 1 E4M3 with gain, 2 E5M2,
 * 3 MXFP4, 4 fused residual add, 5 NVFP4 and statistic 0 none, 1 RMS, 2 MX estimate, 3 post-round estimate.
 * The walk also covers the backward: every row length it accepts, with and without gain and gain gradient, must have
 * a launch plan whose kernel variant exists and whose shared memory fits (first case code -(1 + 2*gain + dgain)).
 * Returns MXN_ERR_NULL when missing_out is NULL and MXN_ERR_SHAPE when max_D < 16. */
mxn_status mxn_selftest_dispatch(int64_t max_D, long long* missing_out, int64_t* first_D_out, int* first_case_out);

/* MXCast - Section 3.2 "Conversion to MXFP8", Eqs. S_tk = cast(m_tk / 256; E8M0),
 * V_tkb = cast(X_tkb / S_tk; E4M3).
 *   x_bf16 [T,D] in; codes_u8 [T,D] out; scales_u8 out (biased E8M0 exponents;
 *   a zero block gets 0). */
mxn_status mx_cast(const void* x_bf16, int64_t T, int64_t D, int block,
                   void* codes_u8, void* scales_u8,
                   mxn_round round, mxn_scale_layout layout, void* cuda_stream);

/* Conventional path, fused - Algorithm 1 "RMSNorm + MXCast", Section 3.1 Eqs. rho_t, Y_td.
 *   r_t = sqrt(mean_d x^2 + eps), rho = 1/r, y = x*rho (then *gain when gain_bf16 [D] is not
 *   NULL), followed by MXCast of y without an intermediate bf16 rounding.
 *   rms_out_or_null [T] fp32 receives r_t (what the backward consumes).
 *   The mean of squares is accumulated in binary32 per thread and binary64 across threads:
 *   r_t agrees with the binary64 definition to about 1e-7 relative, not bit for bit. */
mxn_status rmsnorm_mxfp8_fwd(const void* x_bf16, const void* gain_bf16_or_null,
                             int64_t T, int64_t D, int block, float eps,
                             void* codes_u8, void* scales_u8, float* rms_out_or_null,
                             mxn_round round, mxn_scale_layout layout, void* cuda_stream);

/* MXNorm - Algorithm 2, Section 3.4 Eqs. m~_tk, rho~_t, S~_tk, V~_tkb.
 *   m_k = block absmax of |x|; G = (1/K sum m_k^p)^(1/p), p in {1, 2};
 *   r~ = coef * G (coef_or_0 == 0 selects the paper's printed constant for (B, p):
 *   0.4185 for B = 32, p = 2); rho~ = 1 / (r~ + eps) (0 when the denominator is 0);
 *   scales from m_k * rho~, codes from x * rho~ / S.
 *   gain_bf16_or_null: NULL is the paper's path (the gain is folded into the next weight,
 *   Section 3.7).  Non-NULL is an extension: rho~ still comes from |x|, but scales and codes
 *   are taken from (x * rho~) * gain.
 *   rms_est_out_or_null [T] fp32 receives r~ (cached for the backward, Section 3.7). */
mxn_status mxnorm_fwd(const void* x_bf16, const void* gain_bf16_or_null,
                      int64_t T, int64_t D, int block, int p, float coef_or_0, float eps,
                      void* codes_u8, void* scales_u8, float* rms_est_out_or_null,
                      mxn_round round, mxn_scale_layout layout, void* cuda_stream);

/* Residual add fused in front of MXNorm.  In a pre-norm transformer block the residual branch is added right
 * before the norm (the paper's layer benchmark, appendix "Full Layer Benchmarks", notes that this add is fused
 * with the norm).  h = bf16(x + residual) (binary32 sum, one round-to-nearest-even to bf16) is written to
 * h_out_bf16 [T, D] - the new residual stream, which may alias x_bf16 or residual_bf16 exactly (in-place) -
 * and MXNorm (mxnorm_fwd without gain, the paper's rounding rule) is applied to h without re-reading it.
 * Pointers 32-byte aligned. */
mxn_status mxnorm_add_fwd(const void* x_bf16, const void* residual_bf16, int64_t T, int64_t D, int block, int p,
                          float coef_or_0, float eps, void* h_out_bf16, void* codes_u8, void* scales_u8,
                          float* rms_est_out_or_null, mxn_scale_layout layout, void* cuda_stream);

/* Post-round MXNorm - appendix "Post-round MXNorm" (the paper's ablation; it reports this variant unstable at
 * 8B parameters): the RMS is estimated from the block absmaxes after rounding them to powers of two,
 *   xbar = (1/K) sum_k 2^floor(log2 m_k),  r~ = f^-1(xbar),  f(sigma) = E[max_i 2^floor(log2 |X_i|)] for a block
 *   of B i.i.d. N(0, sigma^2) values; f^-1 by linear interpolation in a table of f^-1(2^(i/64)), i = 0..64, on
 *   [1,2] and f^-1(x) = 2^-k f^-1(2^k x) elsewhere (the table size is this library's choice).
 * Scales and codes then follow mxnorm_fwd with this r~ (no gain, the paper's rounding rule, B in {16,32,64}).
 * The first call for a block size on a device computes the table on the host (tens of milliseconds) and copies
 * it to constant memory - a synchronous copy: make that call outside stream capture. */
mxn_status mxnorm_postround_fwd(const void* x_bf16, int64_t T, int64_t D, int block, float eps,
                                void* codes_u8, void* scales_u8, float* rms_est_out_or_null,
                                mxn_scale_layout layout, void* cuda_stream);

/* NVFP4 variant of MXNorm (the paper benchmarks "B = 16, E2M1" in Section 4.3 but does not
 * define the scale rule; this is the usual NVFP4 convention).
 *   B = 16; r~ and rho~ as in mxnorm_fwd with the (16, p) constant (0.4688 for p = 2);
 *   block scale = E4M3(m_k * rho~ / 6 * global_scale) stored as one E4M3 byte per block
 *   ([T, D/16], row-major or tiled as above); codes = E2M1(x * rho~ * global_scale / scale),
 *   two per byte, element 2i in the low nibble: codes_u8_packed [T, D/2], 8-byte aligned.
 *   Dequantisation: value = code * scale / global_scale.  global_scale = 1 is safe because
 *   MXNorm's output is bounded by sqrt(K)/coef (Lemma 2). */
mxn_status mxnorm_nvfp4_fwd(const void* x_bf16, int64_t T, int64_t D,
                            int p, float coef_or_0, float eps, float global_scale,
                            void* codes_u8_packed, void* scales_e4m3, float* rms_est_out_or_null,
                            mxn_scale_layout layout, void* cuda_stream);

/* The conventional path in the NVFP4 format (Algorithm 1's rho from the true RMS, then the same NVFP4 cast as
 * mxnorm_nvfp4_fwd) - the baseline mxnorm_nvfp4_fwd is compared with, as rmsnorm_mxfp8_fwd is for mxnorm_fwd.
 * Same buffers and conventions as mxnorm_nvfp4_fwd; rms_out_or_null receives sqrt(mean x^2 + eps). */
mxn_status rmsnorm_nvfp4_fwd(const void* x_bf16, int64_t T, int64_t D, float eps, float global_scale,
                             void* codes_u8_packed, void* scales_e4m3, float* rms_out_or_null,
                             mxn_scale_layout layout, void* cuda_stream);

/* The NVFP4 cast without a normaliser (rho = 1), e.g. for the weight operand W*gamma of MXNormLinear in the NVFP4
 * configuration (Section 3.7; the paper does not define NVFP4 beyond block 16 / E2M1, see mxnorm_nvfp4_fwd):
 * block scale = E4M3(absmax / 6 * global_scale), codes = E2M1(x * global_scale / scale).
 * Same buffers and conventions as mxnorm_nvfp4_fwd. */
mxn_status mx_cast_nvfp4(const void* x_bf16, int64_t T, int64_t D, float global_scale,
                      void* codes_u8_packed, void* scales_e4m3, mxn_scale_layout layout, void* cuda_stream);

/* MXFP4 counterparts of the three forward entry points: E2M1 element values (two per byte, element 2i in
 * the low nibble: codes_u8_packed [T, D/2], 32-byte aligned) with E8M0 block scales, B in {16, 32, 64} -
 * the paper's cast with the element type set to E2M1 (appendix "Implementation of MXNormLinear";
 * the kernel benchmark of Section 4.3 covers block sizes {16, 32, 64} x {E4M3, E2M1}).  The largest power
 * of two of E2M1 is 4, so S = 2^(ceil(log2 absmax) - 2) (the paper's rounding rule; no other mode) and
 * codes = E2M1(value / S), round-to-nearest-even, saturating at +-6.  No gain argument. */
mxn_status mx_cast_fp4(const void* x_bf16, int64_t T, int64_t D, int block,
                       void* codes_u8_packed, void* scales_u8, mxn_scale_layout layout, void* cuda_stream);
mxn_status rmsnorm_mxfp4_fwd(const void* x_bf16, int64_t T, int64_t D, int block, float eps,
                             void* codes_u8_packed, void* scales_u8, float* rms_out_or_null,
                             mxn_scale_layout layout, void* cuda_stream);
mxn_status mxnorm_mxfp4_fwd(const void* x_bf16, int64_t T, int64_t D, int block, int p, float coef_or_0, float eps,
                            void* codes_u8_packed, void* scales_u8, float* rms_est_out_or_null,
                            mxn_scale_layout layout, void* cuda_stream);

/* Column-wise (transposed) MXCast for the weight-gradient GEMM of MXNormLinear - Section 3.7,
 * grad W = MXCast(grad H^T) MXCast(rho~ X) gamma: the forward's MX tensor is block-quantised along the hidden
 * axis and cannot be reused, so the activation is re-quantised along the TOKEN axis from the cached X and r~.
 *   y_td = x_td * rho_t with rho_t = 1 / (rms_or_null[t] + eps) (0 when the denominator is 0), or y = x when
 *   rms_or_null is NULL (e.g. for the upstream gradient).  Blocks are 32 consecutive tokens of one column;
 *   S and codes as in mx_cast.  Outputs are laid out transposed: codes_t_u8 [D, T] (32-byte aligned),
 *   scales_t_u8 [D, T/32] row-major or tiled with D as the row index (mxn_scale_bytes(D, T/32, layout)).
 *   Requires T % 32 == 0 and D % 4 == 0; x 8-byte aligned.  The fast kernel (rows staged in shared memory with
 *   16-byte copies, output written in whole 128-byte lines) runs when D % 8 == 0 and x is 16-byte aligned; any
 *   other valid input takes a slower register-only kernel with 8-byte loads. */
mxn_status mx_cast_transposed(const void* x_bf16, const float* rms_or_null, int64_t T, int64_t D, float eps,
                              void* codes_t_u8, void* scales_t_u8,
                              mxn_round round, mxn_scale_layout layout, void* cuda_stream);

/* E5M2 casts for gradient tensors (the paper names E4M3 or E5M2 for gradients in the caption of its
 * computational-graph figure).  OCP E5M2: bias 15, largest finite 57344, largest power of two 2^15, so
 * S = 2^(ceil(log2 absmax) - 15); codes round-to-nearest-even, saturating; E8M0 scales.  Same buffers,
 * alignment and layouts as mx_cast / mx_cast_transposed (no normaliser, the paper's rounding rule only). */
mxn_status mx_cast_e5m2(const void* x_bf16, int64_t T, int64_t D, int block,
                        void* codes_u8, void* scales_u8, mxn_scale_layout layout, void* cuda_stream);
mxn_status mx_cast_transposed_e5m2(const void* x_bf16, int64_t T, int64_t D,
                                   void* codes_t_u8, void* scales_t_u8, mxn_scale_layout layout, void* cuda_stream);

/* Backward - appendix "RMSNorm gradients", used as a straight-through estimator for MXNorm
 * (Section 3.7): the RMSNorm gradient evaluated with the r the forward saved (r~ from
 * mxnorm_fwd, or the true RMS from rmsnorm_mxfp8_fwd - same formula).
 *   grad_out_bf16 [T,D] = dL/dZ with Z = (X / r) * gain;
 *   h = grad_out * gain; delta_t = mean_d(h * x);
 *   dx = h / r - x * delta / r^3        -> dx [T,D], bf16 (dx_is_fp32 == 0) or fp32;
 *   dgain_j = sum_t (x_tj / r_t) * grad_out_tj -> dgain_f32_or_null [D] fp32.
 *   A row with r_t == 0 (a row of zeros, e.g. a padding token: the forward saved r~ = 0 and emitted zeros) gets
 *   dx = 0 and adds nothing to dgain.
 *   Row sums in binary32; the column sum is a deterministic two-stage reduction through
 *   `workspace` (device memory, >= mxnorm_bwd_workspace_bytes(T, D) bytes, 16-byte aligned;
 *   contents on entry irrelevant, clobbered on exit; may be NULL when dgain is NULL).  The size does not
 *   decrease with T: a workspace sized for T rows also serves every call with fewer rows of the same D. */
mxn_status mxnorm_bwd(const void* x_bf16, const void* grad_out_bf16, const void* gain_bf16_or_null,
                      const float* rms, int64_t T, int64_t D,
                      void* dx, int dx_is_fp32, float* dgain_f32_or_null,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t mxnorm_bwd_workspace_bytes(int64_t T, int64_t D);

/* mxnorm_bwd for callers that cannot provide a workspace (the paper has no counterpart; this is a
 * convenience of this library).  Meant for code that may not allocate device memory where it runs:
 * an op inside a framework's fixed memory plan, a plug-in that is handed only the op's tensors, a
 * thread that must stay away from the allocator while another stream is being captured.
 *   Same arguments and results as mxnorm_bwd minus the workspace.  The partial sums of dgain go to
 *   an array built into the library's device image: mxnorm_bwd_noalloc_max_scratch_bytes() = 8 MiB,
 *   reserved on every GPU that loads the library until the process exits.  The call needs
 *   mxnorm_bwd_workspace_bytes(T, D) of it; if that is more (for example D = 16384 with T > 128),
 *   it returns MXN_ERR_TOO_LARGE and enqueues nothing.  With dgain == NULL no scratch is used and any
 *   supported size is accepted.
 *   The first call on each device (with that device current) looks up the array's device address;
 *   make that first call outside any stream capture.  No call allocates or frees memory.
 *   All calls on a device share the one array.  It keeps whatever the previous call left; every
 *   call rewrites the part it reads, so nothing has to be cleared.  Two calls whose kernels may
 *   overlap on the GPU (different streams, no ordering between them) race on it and give wrong
 *   dgain: order such calls, or use mxnorm_bwd with separate workspaces. */
mxn_status mxnorm_bwd_noalloc(const void* x_bf16, const void* grad_out_bf16, const void* gain_bf16_or_null,
                              const float* rms, int64_t T, int64_t D,
                              void* dx, int dx_is_fp32, float* dgain_f32_or_null, void* cuda_stream);
size_t mxnorm_bwd_noalloc_max_scratch_bytes(void);

/* End-to-end convenience for callers whose activations live in HOST memory: mxnorm_fwd (Algorithm 2,
 * no gain) with the host<->device copies inside the call.
 *   x_host_bf16 [T,D], codes_host [T,D], scales_host (mxn_scale_bytes), rms_est_host_or_null [T]
 *   are HOST pointers (pinned memory for asynchronous copies; pageable memory works but serialises).
 *   workspace is DEVICE memory of at least mxnorm_fwd_host_workspace_bytes(T, D, block, layout) bytes,
 *   256-byte aligned, used as staging.  Rows are processed in chunks: the host-to-device copy of chunk
 *   i+1, the kernel of chunk i and the device-to-host copy of chunk i-1 overlap on two internal
 *   non-blocking streams (created on the first call on each device - make that call outside any
 *   stream capture), ordered after prior work on `cuda_stream` and joined back into it.
 *   The call returns once everything is enqueued; the outputs are valid after `cuda_stream` is
 *   synchronised.  No device memory is allocated.  Calls on one device share the internal streams: they are
 *   serialised by a lock while they enqueue (thread-safe, but two host threads do not overlap their pipelines).
 *   If a step fails after work has been enqueued, the caller's stream is still joined with the internal streams
 *   before the error is returned, so buffers may be reused once `cuda_stream` has been synchronised. */
mxn_status mxnorm_fwd_host(const void* x_host_bf16, int64_t T, int64_t D, int block, int p, float coef_or_0,
                           float eps, void* codes_host, void* scales_host, float* rms_est_host_or_null,
                           mxn_round round, mxn_scale_layout layout,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t mxnorm_fwd_host_workspace_bytes(int64_t T, int64_t D, int block, mxn_scale_layout layout);

#ifdef __cplusplus
}
#endif
#endif /* MXNORM_H_ */
