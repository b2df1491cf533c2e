// Register-staged per-block second-moment accumulation (the fall-back of moments_stream.cu) and the
// host entry of the calibration call (Algorithm 2, RTN case, first line
// of the loop):  S_c += sum_t x_{t,c}^T x_{t,c}  for every block c of g channels.
//
// This is a batched SYRK with a tiny output (g x g per block) and a long contraction over
// tokens, i.e. bound by reading Xc once from HBM.  Each warp owns one 32-channel super-block
// and a token range; it loads 16-byte row pieces straight into registers, transposes the 8x8
// sub-tiles with movmatrix so that tokens become the MMA contraction index, and accumulates
// the 32x32 outer-product sum with mma.sync (bf16 products are exact in fp32).  Token ranges
// are split over CTAs; the per-split partial sums go to a workspace and a second kernel adds
// them in a fixed order, so the result does not depend on scheduling.
#include <mutex>

#include "../../include/wush.h"
#include "wush_device.cuh"
#include "wush_host.h"

namespace wush {

constexpr int kMomWarps = 8;      // 8 super-blocks = 256 channels per CTA

template <int G>
__global__ void __launch_bounds__(kMomWarps * 32)
moments_partial_kernel(const __nv_bfloat16* __restrict__ X, int64_t B, int64_t K,
                       float* __restrict__ partials, int tokens_per_split) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int64_t sb = (int64_t)blockIdx.x * kMomWarps + warp;
  if (sb * 32 >= K) return;
  const int64_t t_begin = (int64_t)blockIdx.y * tokens_per_split;
  const int64_t t_end = min(B, t_begin + tokens_per_split);

  float acc[2][4][4];
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b][0] = acc[a][b][1] = acc[a][b][2] = acc[a][b][3] = 0.f;

  const __nv_bfloat16* col = X + sb * 32 + 8 * tig;
  constexpr int UNROLL = 8;
  for (int64_t t0 = t_begin; t0 < t_end; t0 += 16 * UNROLL) {
    uint4 lo[UNROLL], hi[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int64_t ra = t0 + 16 * u + gid, rb = ra + 8;
      lo[u] = (ra < t_end) ? ld_global_nc_v4(col + ra * K) : make_uint4(0, 0, 0, 0);
      hi[u] = (rb < t_end) ? ld_global_nc_v4(col + rb * K) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      // after the transpose register r of a lane holds (tokens 2*tig, 2*tig+1 ; channel
      // 8*(gid/2) + 2*r + gid%2) of the 8-token group
      uint32_t l[4] = {movmatrix_trans(lo[u].x), movmatrix_trans(lo[u].y), movmatrix_trans(lo[u].z),
                       movmatrix_trans(lo[u].w)};
      uint32_t h[4] = {movmatrix_trans(hi[u].x), movmatrix_trans(hi[u].y), movmatrix_trans(hi[u].z),
                       movmatrix_trans(hi[u].w)};
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
          mma_bf16_16816(acc[mt][nt], l[2 * mt], l[2 * mt + 1], h[2 * mt], h[2 * mt + 1], l[nt], h[nt]);
    }
  }

  // acc[mt][nt]: rows i = 8*(gid/2) + 4*mt + gid%2 (+2 for the upper half), cols j = 8*tig + 2*nt (+1)
  const int64_t C = K / G;
  float* out = partials + (int64_t)blockIdx.y * C * G * G;
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int i = 8 * (gid >> 1) + 4 * mt + (gid & 1) + 2 * half;
        const int j = 8 * tig + 2 * nt;
        const float2 v = make_float2(acc[mt][nt][2 * half], acc[mt][nt][2 * half + 1]);
        if (G == 32) {
          *reinterpret_cast<float2*>(out + (sb * 32 + i) * 32 + j) = v;
        } else if ((i >> 4) == (j >> 4)) {
          const int64_t c = sb * 2 + (i >> 4);
          *reinterpret_cast<float2*>(out + (c * 16 + (i & 15)) * 16 + (j & 15)) = v;
        }
      }
}

__global__ void moments_reduce_kernel(const float* __restrict__ partials, int splits, int64_t n,
                                      float* __restrict__ moments, int64_t* __restrict__ count, int64_t B) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i == 0 && count != nullptr) *count += B;
  if (i >= n) return;
  float s = 0.f;
  for (int p = 0; p < splits; ++p) s += partials[(int64_t)p * n + i];
  moments[i] += s;
}

// Sets of partial sums a call needs room for: what the streaming kernel may write per panel (the register-staged
// kernel below takes any number of token splits and is given the same).
int moments_splits(int64_t B, int64_t K) { return moments_stream_segments(B, K); }

cudaError_t run_calib_moments(const void* Xc, int64_t B, int64_t K, int g, float* moments,
                              int64_t* count, float* partials, int splits, cudaStream_t st) {
  // streaming kernel first (TMA-fed ring, ldmatrix.trans operands); it declines when the workspace holds fewer
  // sets of partial sums than it may need, or without the tensor-map driver entry point
  const cudaError_t es = run_calib_moments_stream(Xc, B, K, g, moments, count, partials, splits, st);
  if (es != cudaErrorNotSupported) return es;
  const int64_t groups = (K / 32 + kMomWarps - 1) / kMomWarps;
  int tokens_per_split = (int)((B + splits - 1) / splits);
  tokens_per_split = (tokens_per_split + 15) / 16 * 16;
  dim3 grid((unsigned)groups, (unsigned)splits);
  const __nv_bfloat16* X = reinterpret_cast<const __nv_bfloat16*>(Xc);
  if (g == 32) moments_partial_kernel<32><<<grid, kMomWarps * 32, 0, st>>>(X, B, K, partials, tokens_per_split);
  else         moments_partial_kernel<16><<<grid, kMomWarps * 32, 0, st>>>(X, B, K, partials, tokens_per_split);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int64_t n = K * g;
  moments_reduce_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(partials, splits, n, moments, count, B);
  return cudaGetLastError();
}

}  // namespace wush

// ------------------------------------------------------------------------------------------
// wush_calib_moments_static: the same computation with the per-split partial sums kept in a
// fixed device array that is part of the library image, for callers that cannot supply
// scratch memory (see include/wush.h).
namespace wush {
namespace {

constexpr size_t kStaticScratchFloats = WUSH_STATIC_SCRATCH_BYTES / sizeof(float);
static __device__ __align__(256) float g_static_partials[kStaticScratchFloats];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
float* g_static_ptr[kMaxDevices] = {};      // device address of g_static_partials, per device

// Resolves the device address of the array on the CURRENT device (once per device).  In host
// code the symbol's name is only a handle; kernels need the address the runtime returns.
cudaError_t static_scratch(float** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_ptr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_partials);
    if (e != cudaSuccess) return e;
    g_static_ptr[dev] = static_cast<float*>(p);
  }
  *out = g_static_ptr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace wush

extern "C" int wush_calib_moments_static(const void* Xc, int64_t B, int64_t K, int g, float* moments,
                                         int64_t* count, void* stream) {
  if (g != 16 && g != 32) return WUSH_ERR_FORMAT;
  if (B < 0 || K <= 0 || K % g != 0 || K % 64 != 0 || B > (int64_t)1 << 30 || K > (int64_t)1 << 30)
    return WUSH_ERR_SHAPE;
  if (!Xc || !moments || !count) return WUSH_ERR_NULL;
  if (((reinterpret_cast<uintptr_t>(Xc) | reinterpret_cast<uintptr_t>(moments)) & 15u) != 0) return WUSH_ERR_ALIGN;
  if ((reinterpret_cast<uintptr_t>(count) & 7u) != 0) return WUSH_ERR_ALIGN;
  const size_t per_split = (size_t)K * (size_t)g;                 // floats of one partial set
  if (per_split > wush::kStaticScratchFloats) return WUSH_ERR_WORKSPACE;   // K * g beyond the built-in scratch
  if (B == 0) return WUSH_OK;
  int splits = wush::moments_splits(B, K);
  const size_t fit = wush::kStaticScratchFloats / per_split;
  if ((size_t)splits > fit) splits = (int)fit;
  float* scratch = nullptr;
  cudaError_t e = wush::static_scratch(&scratch);
  if (e != cudaSuccess) return wush::record_cuda_error(e, "address of the built-in scratch array");
  e = wush::run_calib_moments(Xc, B, K, g, moments, count, scratch, splits, (cudaStream_t)stream);
  return e == cudaSuccess ? WUSH_OK : wush::record_cuda_error(e);
}
