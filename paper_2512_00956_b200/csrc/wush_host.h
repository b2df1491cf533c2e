// Internal host-side declarations of libwush (not part of the public ABI).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace wush {

// One-time launch set-up (function attributes, SM count, cluster occupancy) is remembered per device: the
// caches below are arrays indexed by the current device.  -1: no usable current device.
constexpr int kDeviceSlots = 64;
inline int device_slot() {
  int d = 0;
  if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= kDeviceSlots) return -1;
  return d;
}

// Optional rules of the activation quantiser.  mx_ceil: MXFP4 exponent by the ceil rule.  amax_in / ts_out
// (NVFP4): take the tensor scale from *amax_in (bit pattern of the AbsMax found by run_act_amax) instead of
// `ts`, and write the scale used to *ts_out.
struct QuantOpts {
  bool mx_ceil = false;
  const uint32_t* amax_in = nullptr;
  float* ts_out = nullptr;
  uint32_t* amax_out = nullptr;   // run_quantize_act_stream only: AbsMax pass instead of quantising (g = 16)
  int drop_item = -1;             // test hook: the producer never requests this work item (streaming kernel only)
  int force_rows = 0;             // test hook: 64 or 128 = tile height of the streaming kernel whatever the problem size
};
// Text of the last CUDA error of the calling thread (wush_last_cuda_error); returns WUSH_ERR_CUDA.
int record_cuda_error(cudaError_t e, const char* why = nullptr);
// clear_status: the kernel zeroes *status itself (wush_linear); otherwise the word is left alone
cudaError_t run_quantize_act(const void* X, int64_t M, int64_t K, const void* T, int g, const float* ts,
                             uint8_t* codes, uint8_t* scales, int sf, int32_t* status, bool clear_status,
                             bool pdl, cudaStream_t st, const QuantOpts& opt = QuantOpts());
// status / clear_status: as for run_quantize_act (the AbsMax pass reports an expired wait in the same word)
cudaError_t run_act_amax(const void* X, int64_t M, int64_t K, const void* T, uint32_t* amax, cudaStream_t st,
                         int32_t* status = nullptr, bool clear_status = false, int force_rows = 0);
// out[0] = NVFP4 tensor scale of the transformed tokens (AbsMax / 2688, 1 if all zero), out[1] = that AbsMax
cudaError_t run_act_tensor_scale(const void* X, int64_t M, int64_t K, const void* T, float* out, cudaStream_t st);
// streaming (TMA-fed, persistent) variant; cudaErrorNotSupported = problem not covered, use the other kernel
cudaError_t run_quantize_act_stream(const void* X, int64_t M, int64_t K, const void* T, int g, const float* ts,
                                    uint8_t* codes, uint8_t* scales, int sf, int32_t* status, bool clear_status,
                                    bool pdl, cudaStream_t st, const QuantOpts& opt = QuantOpts());
// activation side with the block products on tcgen05 tensor cores (transform_quant_tc.cu); same contract
cudaError_t run_quantize_act_tc(const void* X, int64_t M, int64_t K, const void* T, int g, const float* ts,
                                uint8_t* codes, uint8_t* scales, int sf, int32_t* status, bool clear_status,
                                bool pdl, cudaStream_t st, const QuantOpts& opt = QuantOpts());
cudaError_t run_quantize_weight_tc(const void* W, int64_t N, int64_t K, const float* Tinv, int g, uint8_t* codes,
                                   uint8_t* scales, int sf, cudaStream_t st, const QuantOpts& opt);
// weight side through the streaming kernel (fp32 Tinv, three-way split); cudaErrorNotSupported = use the other kernel
cudaError_t run_quantize_weight_stream(const void* W, int64_t N, int64_t K, const float* Tinv, int g, uint8_t* codes,
                                       uint8_t* scales, int sf, cudaStream_t st, const QuantOpts& opt);
cudaError_t run_transform_f32(const void* X, int64_t M, int64_t K, const void* T, int g, bool t_is_f32,
                              float* V, cudaStream_t st);
cudaError_t run_quantize_weight(const void* W, int64_t N, int64_t K, const float* Tinv, int g,
                                float* ts_out, uint8_t* codes, uint8_t* scales, int sf,
                                uint32_t* amax_ws, cudaStream_t st, bool mx_ceil = false, int force_rows = 0);
cudaError_t run_quantize_f32(const float* V, int64_t R, int64_t K, int g, const float* ts,
                             uint8_t* codes, uint8_t* scales, int sf, cudaStream_t st, bool mx_ceil = false);

cudaError_t run_check_division(const float* divisors, int n, unsigned long long* mismatches, cudaStream_t st);

int moments_splits(int64_t B, int64_t K);
int moments_stream_segments(int64_t B, int64_t K);
// streaming moments (partial sums + segment-aware reduction); cudaErrorNotSupported = use the other kernels
cudaError_t run_calib_moments_stream(const void* Xc, int64_t B, int64_t K, int g, float* moments, int64_t* count,
                                     float* partials, int slots, cudaStream_t st);
cudaError_t run_calib_moments(const void* Xc, int64_t B, int64_t K, int g, float* moments,
                              int64_t* count, float* partials, int splits, cudaStream_t st);

// Block-scaled FP4 GEMM.  Returns cudaSuccess or the failing CUDA error; `why` (optional)
// receives a static description when the failure is not a CUDA error (e.g. no driver symbol).
cudaError_t run_gemm_fp4(const uint8_t* Xq, const uint8_t* Xs, const uint8_t* Wq, const uint8_t* Ws,
                         int64_t M, int64_t N, int64_t K, int fmt, const float* tsx, const float* tsw,
                         void* Y, int out_bf16, int32_t* status, bool clear_status, bool after_quantizer, cudaStream_t st,
                         const char** why);

cudaError_t run_build_transforms(const float* mom_w, int64_t n_w, const float* mom_x, int64_t n_x, int64_t K, int g,
                                 double lambda, void* T, float* Tinv, int32_t* info, cudaStream_t st,
                                 bool with_hadamard = true);
cudaError_t run_invert_transforms(const void* T, int64_t K, int g, float* Tinv, int32_t* info, cudaStream_t st);
// kind 0: one shared normalised Hadamard matrix, kind 1: the identity, for every block; Tinv = T^-T of the stored values
cudaError_t run_fixed_transforms(int kind, int64_t K, int g, void* T, float* Tinv, int32_t* info, cudaStream_t st);

cudaError_t run_build_transform_f64(const double* mom_w, double inv_nw, const double* mom_x, double inv_nx, int g,
                                    double lambda, void* T, float* Tinv, int32_t* info, cudaStream_t st);
// Algorithm 2, GPTQ case (gptq.cu).  ts_w: NVFP4 weight tensor scale (device, input) or nullptr.
size_t gptq_workspace_bytes(int64_t N, int64_t K, int g);
cudaError_t run_gptq_quantize_weight(const void* W, int64_t N, int64_t K, const void* Xc, int64_t B, int fmt, int g,
                                     double lambda, const float* ts_w, void* T, float* Tinv, uint8_t* codes,
                                     uint8_t* scales, int sf, int32_t* info, void* workspace, int mx_ceil, cudaStream_t st);

// two-CTA persistent variant (M > 128); cudaErrorNotSupported = use the single-CTA kernel
int gemm_2cta_cluster_limit(int clusters);   // test hook: 0 = no limit; returns the previous value (per device)
cudaError_t run_gemm_fp4_2cta(const uint8_t* Xq, const uint8_t* Xs, const uint8_t* Wq, const uint8_t* Ws, int64_t M,
                              int64_t N, int64_t K, int fmt, const float* tsx, const float* tsw, void* Y,
                              int out_bf16, int32_t* status, bool clear_status, bool pdl, cudaStream_t st);

}  // namespace wush
