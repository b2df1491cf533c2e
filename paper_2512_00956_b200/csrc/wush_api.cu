// extern "C" entry points of libwush: argument validation and dispatch.  See include/wush.h
// for the contract of every call.
#include <stdio.h>
#include <string.h>

#include <atomic>

#include "../../include/wush.h"
#include "wush_device.cuh"
#include "wush_host.h"

namespace {
thread_local char g_cuda_error[256] = "";
}

int wush::record_cuda_error(cudaError_t e, const char* why) {
  snprintf(g_cuda_error, sizeof(g_cuda_error), "%s%s%s", cudaGetErrorString(e), why ? ": " : "", why ? why : "");
  return WUSH_ERR_CUDA;
}

namespace {

inline int cuda_fail(cudaError_t e, const char* why = nullptr) { return wush::record_cuda_error(e, why); }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int check_fmt(int fmt, int g) {
  if (fmt == WUSH_MXFP4 || fmt == WUSH_MXFP4_CEIL) return g == 32 ? WUSH_OK : WUSH_ERR_FORMAT;
  if (fmt == WUSH_NVFP4) return g == 16 ? WUSH_OK : WUSH_ERR_FORMAT;
  return WUSH_ERR_FORMAT;
}
inline int check_shape(int64_t rows, int64_t K, int g) {
  if (rows < 0 || K <= 0 || g <= 0) return WUSH_ERR_SHAPE;
  if (K % g != 0 || K % 64 != 0) return WUSH_ERR_SHAPE;
  if (rows > (int64_t)1 << 30 || K > (int64_t)1 << 30) return WUSH_ERR_SHAPE;
  return WUSH_OK;
}
inline size_t round16(size_t x) { return (x + 15) & ~size_t(15); }
// the GEMM knows two formats; the scale rule only matters to the quantisers
inline int gemm_fmt(int fmt) { return fmt == WUSH_NVFP4 ? wush::kFmtNV : wush::kFmtMX; }

// test hook (wush_debug_drop_tile): work item + 1 that the next streaming-quantiser launch of wush_linear on this
// device will not load (0 = none); one shot, taken with an atomic exchange so that concurrent callers cannot
// both consume it
std::atomic<int> g_drop_item[wush::kDeviceSlots];
int take_drop_item() {
  const int slot = wush::device_slot();
  if (slot < 0) return -1;
  return g_drop_item[slot].exchange(0) - 1;
}
// test hook (wush_debug_quantiser_rows): forced tile height of the streaming quantiser on this device (0 = automatic)
std::atomic<int> g_force_rows[wush::kDeviceSlots];
int forced_rows() {
  const int slot = wush::device_slot();
  return slot < 0 ? 0 : g_force_rows[slot].load();
}

inline wush::QuantOpts opts_of(int fmt) {
  wush::QuantOpts o;
  o.mx_ceil = (fmt == WUSH_MXFP4_CEIL);
  o.force_rows = forced_rows();
  return o;
}

bool device_is_sm100() {
  static signed char cached[wush::kDeviceSlots] = {};   // 0 unknown, 1 yes, -1 no; per device
  const int slot = wush::device_slot();
  if (slot < 0) return false;
  if (cached[slot] == 0) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, slot) != cudaSuccess) return false;
    cached[slot] = (major == 10) ? 1 : -1;
  }
  return cached[slot] == 1;
}

}  // namespace

extern "C" {

const char* wush_status_string(int status) {
  switch (status) {
    case WUSH_OK: return "ok";
    case WUSH_ERR_NULL: return "null pointer";
    case WUSH_ERR_SHAPE: return "bad shape";
    case WUSH_ERR_FORMAT: return "bad format / group size / layout";
    case WUSH_ERR_ALIGN: return "pointer not 16-byte aligned";
    case WUSH_ERR_WORKSPACE: return "workspace missing or too small";
    case WUSH_ERR_CUDA: return "CUDA error";
    case WUSH_ERR_TIMEOUT: return "bounded device wait expired";
    case WUSH_ERR_DEVICE: return "device is not compute capability 10.x";
    default: return "unknown status";
  }
}

const char* wush_last_cuda_error(void) { return g_cuda_error; }

size_t wush_scale_bytes(int64_t rows, int64_t K, int g, wush_sf_layout_t sf) {
  if (rows < 0 || K <= 0 || (g != 16 && g != 32) || K % g != 0) return 0;
  const int64_t KB = K / g;
  if (sf == WUSH_SF_LINEAR) return (size_t)(rows * KB);
  if (sf == WUSH_SF_TILED) return (size_t)(((rows + 127) / 128) * ((KB + 3) / 4) * 512);
  return 0;
}

int wush_quantize_act(const void* X, int64_t M, int64_t K, const void* T, wush_format_t fmt, int g,
                      const float* x_tensor_scale, uint8_t* codes, uint8_t* scales, wush_sf_layout_t sf,
                      void* stream) {
  int rc = check_fmt(fmt, g);
  if (rc) return rc;
  if ((rc = check_shape(M, K, g))) return rc;
  if (sf != WUSH_SF_LINEAR && sf != WUSH_SF_TILED) return WUSH_ERR_FORMAT;
  if (!X || !T || !codes || !scales || (fmt == WUSH_NVFP4 && !x_tensor_scale)) return WUSH_ERR_NULL;
  if (!aligned16(X) || !aligned16(T) || !aligned16(codes) || !aligned16(scales)) return WUSH_ERR_ALIGN;
  if (M == 0) return WUSH_OK;
  cudaError_t e = wush::run_quantize_act(X, M, K, T, g, x_tensor_scale, codes, scales, (int)sf, nullptr, false, false,
                                         (cudaStream_t)stream, opts_of(fmt));
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e);
}

int wush_quantize_act_dynamic(const void* X, int64_t M, int64_t K, const void* T, int g, float* x_tensor_scale,
                              uint8_t* codes, uint8_t* scales, wush_sf_layout_t sf, void* stream) {
  int rc = check_fmt(WUSH_NVFP4, g);
  if (rc) return rc;
  if ((rc = check_shape(M, K, g))) return rc;
  if (sf != WUSH_SF_LINEAR && sf != WUSH_SF_TILED) return WUSH_ERR_FORMAT;
  if (!X || !T || !codes || !scales || !x_tensor_scale) return WUSH_ERR_NULL;
  if (!aligned16(X) || !aligned16(T) || !aligned16(codes) || !aligned16(scales)) return WUSH_ERR_ALIGN;
  if ((reinterpret_cast<uintptr_t>(x_tensor_scale) & 7u) != 0) return WUSH_ERR_ALIGN;
  if (M == 0) return WUSH_OK;
  uint32_t* amax = reinterpret_cast<uint32_t*>(x_tensor_scale + 1);
  cudaError_t e = wush::run_act_amax(X, M, K, T, amax, (cudaStream_t)stream, nullptr, false, forced_rows());
  if (e != cudaSuccess) return cuda_fail(e);
  wush::QuantOpts o = opts_of(WUSH_NVFP4);
  o.amax_in = amax;
  o.ts_out = x_tensor_scale;
  e = wush::run_quantize_act(X, M, K, T, g, nullptr, codes, scales, (int)sf, nullptr, false, false, (cudaStream_t)stream, o);
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e);
}

int wush_act_tensor_scale(const void* Xc, int64_t B, int64_t K, const void* T, int g, float* out, void* stream) {
  int rc = check_fmt(WUSH_NVFP4, g);
  if (rc) return rc;
  if ((rc = check_shape(B, K, g))) return rc;
  if (!Xc || !T || !out) return WUSH_ERR_NULL;
  if (!aligned16(Xc) || !aligned16(T) || (reinterpret_cast<uintptr_t>(out) & 7u) != 0) return WUSH_ERR_ALIGN;
  if (B == 0) return WUSH_ERR_SHAPE;
  const cudaError_t e = wush::run_act_tensor_scale(Xc, B, K, T, out, (cudaStream_t)stream);
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e);
}

size_t wush_quantize_weight_workspace_bytes(int64_t, int64_t, wush_format_t, int) { return 256; }

int wush_quantize_weight(const void* W, int64_t N, int64_t K, const float* Tinv, wush_format_t fmt, int g,
                         float* w_tensor_scale, uint8_t* codes, uint8_t* scales, wush_sf_layout_t sf,
                         void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_fmt(fmt, g);
  if (rc) return rc;
  if ((rc = check_shape(N, K, g))) return rc;
  if (sf != WUSH_SF_LINEAR && sf != WUSH_SF_TILED) return WUSH_ERR_FORMAT;
  if (!W || !Tinv || !codes || !scales || (fmt == WUSH_NVFP4 && !w_tensor_scale)) return WUSH_ERR_NULL;
  if (!workspace || workspace_bytes < wush_quantize_weight_workspace_bytes(N, K, fmt, g)) return WUSH_ERR_WORKSPACE;
  if (!aligned16(W) || !aligned16(Tinv) || !aligned16(codes) || !aligned16(scales) || !aligned16(workspace))
    return WUSH_ERR_ALIGN;
  if (N == 0) return WUSH_OK;
  cudaError_t e = wush::run_quantize_weight(W, N, K, Tinv, g, w_tensor_scale, codes, scales, (int)sf,
                                            reinterpret_cast<uint32_t*>(workspace), (cudaStream_t)stream,
                                            fmt == WUSH_MXFP4_CEIL, forced_rows());
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e);
}

int wush_gemm_fp4(const uint8_t* Xq, const uint8_t* Xs, const uint8_t* Wq, const uint8_t* Ws, int64_t M,
                  int64_t N, int64_t K, wush_format_t fmt, int g, const float* x_tensor_scale,
                  const float* w_tensor_scale, void* Y, wush_out_t ydt, int32_t* status, void* stream) {
  int rc = check_fmt(fmt, g);
  if (rc) return rc;
  if ((rc = check_shape(M, K, g))) return rc;
  if (N <= 0 || N % 8 != 0 || N > (int64_t)1 << 30) return WUSH_ERR_SHAPE;
  if (ydt != WUSH_OUT_F32 && ydt != WUSH_OUT_BF16) return WUSH_ERR_FORMAT;
  if (!Xq || !Xs || !Wq || !Ws || !Y) return WUSH_ERR_NULL;
  if (fmt == WUSH_NVFP4 && (!x_tensor_scale || !w_tensor_scale)) return WUSH_ERR_NULL;
  if (!aligned16(Xq) || !aligned16(Xs) || !aligned16(Wq) || !aligned16(Ws) || !aligned16(Y)) return WUSH_ERR_ALIGN;
  if (M == 0) return WUSH_OK;
  if (!device_is_sm100()) return WUSH_ERR_DEVICE;
  const char* why = nullptr;
  cudaError_t e = wush::run_gemm_fp4(Xq, Xs, Wq, Ws, M, N, K, gemm_fmt(fmt), x_tensor_scale, w_tensor_scale, Y,
                                     ydt == WUSH_OUT_BF16, status, true, false, (cudaStream_t)stream, &why);
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e, why);
}

size_t wush_linear_workspace_bytes(int64_t M, int64_t K, int g) {
  if (M < 0 || K <= 0 || (g != 16 && g != 32) || K % g != 0) return 0;
  // packed codes | TILED scale bytes | fp32 tensor scale + AbsMax (per-batch NVFP4 scale) | status word
  return round16((size_t)(M * (K / 2))) + round16(wush_scale_bytes(M, K, g, WUSH_SF_TILED)) + 16 + 16;
}

size_t wush_workspace_bytes(int64_t M, int64_t N, int64_t K, wush_format_t fmt, int g) {
  if (check_fmt(fmt, g) != WUSH_OK || M < 0 || N < 0 || K <= 0 || K % g != 0) return 0;
  size_t need = wush_linear_workspace_bytes(M, K, g);
  const size_t wq = wush_quantize_weight_workspace_bytes(N, K, fmt, g);
  const size_t mom = wush_calib_moments_workspace_bytes(M > N ? M : N, K, g);
  if (wq > need) need = wq;
  if (mom > need) need = mom;
  return need;
}

int wush_linear(const void* X, int64_t M, int64_t K, const void* T, const uint8_t* Wcodes,
                const uint8_t* Wscales, int64_t N, const float* x_tensor_scale, const float* w_tensor_scale,
                wush_format_t fmt, int g, void* Y, wush_out_t ydt, void* workspace, size_t workspace_bytes,
                void* stream) {
  int rc = check_fmt(fmt, g);
  if (rc) return rc;
  if ((rc = check_shape(M, K, g))) return rc;
  if (!workspace || workspace_bytes < wush_linear_workspace_bytes(M, K, g)) return WUSH_ERR_WORKSPACE;
  if (!aligned16(workspace)) return WUSH_ERR_ALIGN;
  uint8_t* xq = reinterpret_cast<uint8_t*>(workspace);
  uint8_t* xs = xq + round16((size_t)(M * (K / 2)));
  float* ts_dyn = reinterpret_cast<float*>(xs + round16(wush_scale_bytes(M, K, g, WUSH_SF_TILED)));
  int32_t* status = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(ts_dyn) + 16);
  const bool dynamic = (fmt == WUSH_NVFP4 && x_tensor_scale == nullptr);
  // validate the GEMM's arguments before the quantiser touches anything
  if (N <= 0 || N % 8 != 0) return WUSH_ERR_SHAPE;
  if (ydt != WUSH_OUT_F32 && ydt != WUSH_OUT_BF16) return WUSH_ERR_FORMAT;
  if (!X || !T || !Wcodes || !Wscales || !Y) return WUSH_ERR_NULL;
  if (fmt == WUSH_NVFP4 && !w_tensor_scale) return WUSH_ERR_NULL;
  if (!aligned16(Wcodes) || !aligned16(Wscales) || !aligned16(Y)) return WUSH_ERR_ALIGN;
  if (!X || !T) return WUSH_ERR_NULL;
  if (!aligned16(X) || !aligned16(T)) return WUSH_ERR_ALIGN;
  if (M == 0) return WUSH_OK;
  if (!device_is_sm100()) return WUSH_ERR_DEVICE;
  // one status word for both kernels: cleared by the quantiser kernel, set by whichever bounded wait expires
  wush::QuantOpts o = opts_of(fmt);
  o.drop_item = take_drop_item();
  cudaError_t e;
  if (dynamic) {                                  // per-batch tensor scale: AbsMax pass first
    uint32_t* amax = reinterpret_cast<uint32_t*>(ts_dyn + 1);
    // the AbsMax pass clears the status word and reports into it; the quantising pass must then leave it alone
    if ((e = wush::run_act_amax(X, M, K, T, amax, (cudaStream_t)stream, status, true, o.force_rows)) != cudaSuccess) return cuda_fail(e);
    o.amax_in = amax;
    o.ts_out = ts_dyn;
    x_tensor_scale = ts_dyn;                      // what the GEMM multiplies by
  }
  e = wush::run_quantize_act(X, M, K, T, g, dynamic ? nullptr : x_tensor_scale, xq, xs, WUSH_SF_TILED, status, !dynamic, true,
                             (cudaStream_t)stream, o);
  if (e != cudaSuccess) return cuda_fail(e);
  const char* why = nullptr;
  e = wush::run_gemm_fp4(xq, xs, Wcodes, Wscales, M, N, K, gemm_fmt(fmt), x_tensor_scale, w_tensor_scale, Y,
                         ydt == WUSH_OUT_BF16, status, false, true, (cudaStream_t)stream, &why);
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e, why);
}

size_t wush_calib_moments_workspace_bytes(int64_t B, int64_t K, int g) {
  if (B < 0 || K <= 0 || (g != 16 && g != 32) || K % g != 0) return 0;
  return (size_t)wush::moments_splits(B, K) * (size_t)K * (size_t)g * sizeof(float);
}

int wush_calib_moments(const void* Xc, int64_t B, int64_t K, int g, float* moments, int64_t* count,
                       void* workspace, size_t workspace_bytes, void* stream) {
  if (g != 16 && g != 32) return WUSH_ERR_FORMAT;
  int rc = check_shape(B, K, g);
  if (rc) return rc;
  if (!Xc || !moments || !count) return WUSH_ERR_NULL;
  if (!workspace || workspace_bytes < wush_calib_moments_workspace_bytes(B, K, g)) return WUSH_ERR_WORKSPACE;
  if (!aligned16(Xc) || !aligned16(moments) || !aligned16(workspace)) return WUSH_ERR_ALIGN;
  if ((reinterpret_cast<uintptr_t>(count) & 7u) != 0) return WUSH_ERR_ALIGN;
  if (B == 0) return WUSH_OK;
  cudaError_t e = wush::run_calib_moments(Xc, B, K, g, moments, count, reinterpret_cast<float*>(workspace),
                                          wush::moments_splits(B, K), (cudaStream_t)stream);
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e);
}

int wush_build_transforms_kind(const float* mom_w, int64_t rows_w, const float* mom_x, int64_t rows_x, int64_t K,
                               int g, float lambda, wush_transform_kind_t kind, void* T, float* Tinv, int32_t* info,
                               void* stream) {
  if (g != 16 && g != 32) return WUSH_ERR_FORMAT;
  if (kind == WUSH_KIND_HADAMARD || kind == WUSH_KIND_IDENTITY) {       // data-independent: the moments are not read
    if (K <= 0 || K % g != 0) return WUSH_ERR_SHAPE;
    if (!T || !Tinv) return WUSH_ERR_NULL;
    if (!aligned16(T) || !aligned16(Tinv)) return WUSH_ERR_ALIGN;
    const cudaError_t ef = wush::run_fixed_transforms(kind == WUSH_KIND_HADAMARD ? 0 : 1, K, g, T, Tinv, info, (cudaStream_t)stream);
    return ef == cudaSuccess ? WUSH_OK : cuda_fail(ef);
  }
  if (kind != WUSH_KIND_WUSH && kind != WUSH_KIND_WUS) return WUSH_ERR_FORMAT;
  if (K <= 0 || K % g != 0 || rows_w <= 0 || rows_x <= 0 || !(lambda >= 0.0f)) return WUSH_ERR_SHAPE;
  if (!mom_w || !mom_x || !T || !Tinv) return WUSH_ERR_NULL;
  if (!aligned16(mom_w) || !aligned16(mom_x) || !aligned16(T) || !aligned16(Tinv)) return WUSH_ERR_ALIGN;
  cudaError_t e = wush::run_build_transforms(mom_w, rows_w, mom_x, rows_x, K, g, (double)lambda, T, Tinv, info,
                                             (cudaStream_t)stream, kind == WUSH_KIND_WUSH);
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e);
}

int wush_build_transforms(const float* mom_w, int64_t rows_w, const float* mom_x, int64_t rows_x, int64_t K, int g,
                          float lambda, void* T, float* Tinv, int32_t* info, void* stream) {
  return wush_build_transforms_kind(mom_w, rows_w, mom_x, rows_x, K, g, lambda, WUSH_KIND_WUSH, T, Tinv, info, stream);
}

size_t wush_gptq_workspace_bytes(int64_t N, int64_t K, int g) {
  if (N <= 0 || K <= 0 || (g != 16 && g != 32) || K % g != 0) return 0;
  return wush::gptq_workspace_bytes(N, K, g);
}

int wush_gptq_quantize_weight(const void* W, int64_t N, int64_t K, const void* Xc, int64_t B, wush_format_t fmt, int g,
                              float lambda, const float* w_tensor_scale, void* T, float* Tinv, uint8_t* codes,
                              uint8_t* scales, wush_sf_layout_t sf, int32_t* info, void* workspace,
                              size_t workspace_bytes, void* stream) {
  int rc = check_fmt(fmt, g);
  if (rc) return rc;
  if ((rc = check_shape(N, K, g))) return rc;
  if (N == 0 || B <= 0 || B > (int64_t)1 << 30 || K > 32768 || !(lambda > 0.0f)) return WUSH_ERR_SHAPE;
  if (sf != WUSH_SF_LINEAR && sf != WUSH_SF_TILED) return WUSH_ERR_FORMAT;
  if (!W || !Xc || !T || !Tinv || !codes || !scales || (fmt == WUSH_NVFP4 && !w_tensor_scale)) return WUSH_ERR_NULL;
  if (!workspace || workspace_bytes < wush_gptq_workspace_bytes(N, K, g)) return WUSH_ERR_WORKSPACE;
  if (!aligned16(W) || !aligned16(Xc) || !aligned16(T) || !aligned16(Tinv) || !aligned16(codes) || !aligned16(scales) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return WUSH_ERR_ALIGN;
  const cudaError_t e = wush::run_gptq_quantize_weight(W, N, K, Xc, B, gemm_fmt(fmt), g, (double)lambda, w_tensor_scale, T, Tinv,
                                                       codes, scales, (int)sf, info, workspace, fmt == WUSH_MXFP4_CEIL ? 1 : 0,
                                                       (cudaStream_t)stream);
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e);
}

int wush_invert_transforms(const void* T, int64_t K, int g, float* Tinv, int32_t* info, void* stream) {
  if (g != 16 && g != 32) return WUSH_ERR_FORMAT;
  if (K <= 0 || K % g != 0) return WUSH_ERR_SHAPE;
  if (!T || !Tinv) return WUSH_ERR_NULL;
  if (!aligned16(T) || !aligned16(Tinv)) return WUSH_ERR_ALIGN;
  cudaError_t e = wush::run_invert_transforms(T, K, g, Tinv, info, (cudaStream_t)stream);
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e);
}

int wush_quantize_f32(const float* V, int64_t R, int64_t K, wush_format_t fmt, int g, const float* tensor_scale,
                      uint8_t* codes, uint8_t* scales, wush_sf_layout_t sf, void* stream) {
  int rc = check_fmt(fmt, g);
  if (rc) return rc;
  if ((rc = check_shape(R, K, g))) return rc;
  if (sf != WUSH_SF_LINEAR && sf != WUSH_SF_TILED) return WUSH_ERR_FORMAT;
  if (!V || !codes || !scales || (fmt == WUSH_NVFP4 && !tensor_scale)) return WUSH_ERR_NULL;
  if (!aligned16(V) || !aligned16(codes) || !aligned16(scales)) return WUSH_ERR_ALIGN;
  if (R == 0) return WUSH_OK;
  cudaError_t e = wush::run_quantize_f32(V, R, K, g, tensor_scale, codes, scales, (int)sf, (cudaStream_t)stream,
                                         fmt == WUSH_MXFP4_CEIL);
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e);
}

int wush_debug_gemm_clusters(int clusters) { return wush::gemm_2cta_cluster_limit(clusters); }

int wush_debug_drop_tile(int item) {
  const int slot = wush::device_slot();
  if (slot < 0) return WUSH_ERR_CUDA;
  g_drop_item[slot].store(item < 0 ? 0 : item + 1);
  return WUSH_OK;
}

int wush_debug_quantiser_rows(int rows) {
  const int slot = wush::device_slot();
  if (slot < 0) return WUSH_ERR_CUDA;
  if (rows != 0 && rows != 64 && rows != 128) return WUSH_ERR_SHAPE;
  return g_force_rows[slot].exchange(rows);
}

int wush_decode_status(int32_t word) { return word == 0 ? WUSH_OK : WUSH_ERR_TIMEOUT; }

int wush_check_division(const float* divisors, int n, uint64_t* mismatches, void* stream) {
  if (n < 0 || n > 65535) return WUSH_ERR_SHAPE;
  if (!divisors || !mismatches) return WUSH_ERR_NULL;
  if (n == 0) return WUSH_OK;
  cudaError_t e = wush::run_check_division(divisors, n, reinterpret_cast<unsigned long long*>(mismatches), (cudaStream_t)stream);
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e);
}

int wush_transform_act_f32(const void* X, int64_t M, int64_t K, const void* T, int g, float* V, void* stream) {
  if (g != 16 && g != 32) return WUSH_ERR_FORMAT;
  int rc = check_shape(M, K, g);
  if (rc) return rc;
  if (!X || !T || !V) return WUSH_ERR_NULL;
  if (!aligned16(X) || !aligned16(T) || !aligned16(V)) return WUSH_ERR_ALIGN;
  if (M == 0) return WUSH_OK;
  cudaError_t e = wush::run_transform_f32(X, M, K, T, g, false, V, (cudaStream_t)stream);
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e);
}

int wush_transform_weight_f32(const void* W, int64_t N, int64_t K, const float* Tinv, int g, float* V,
                              void* stream) {
  if (g != 16 && g != 32) return WUSH_ERR_FORMAT;
  int rc = check_shape(N, K, g);
  if (rc) return rc;
  if (!W || !Tinv || !V) return WUSH_ERR_NULL;
  if (!aligned16(W) || !aligned16(Tinv) || !aligned16(V)) return WUSH_ERR_ALIGN;
  if (N == 0) return WUSH_OK;
  cudaError_t e = wush::run_transform_f32(W, N, K, Tinv, g, true, V, (cudaStream_t)stream);
  return e == cudaSuccess ? WUSH_OK : cuda_fail(e);
}

}  // extern "C"
