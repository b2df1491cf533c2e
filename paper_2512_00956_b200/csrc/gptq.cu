// Algorithm 2, GPTQ case ("Compute WUSH and Pre-Quantize Weights"): WUSH transforms built from the UPDATED
// weights, interleaved with GPTQ's error propagation.  An offline solver, sequential over the d_in / d blocks;
// everything is fp64 on the device, one plain kernel per step - correctness and parity with the CPU oracle come
// first here, this is not a roofline kernel.
//
// Row-major view of the paper's column-vector notation: W[N][K] (N = d_out rows, K = d_in columns), block (i) is
// columns i*d .. i*d + d - 1.  Steps, in the paper's order:
//   H      = Xc^T Xc / B                                (GPTQ's Hessian, K x K)
//   M_X(i) = diagonal blocks of H
//   L L^T  = (H + lambda * tr(H)/K * I)^-1              (L lower).  Computed without forming the inverse: with the
//            factorisation Hd = U U^T, U UPPER triangular, Hd^-1 = U^-T U^-1, so L = (U^-1)^T.  V = U^-1 is kept
//            (upper triangular); L[r][c] = V[c][r].
//   for i = 0 .. K/d - 1:
//     M_W(i)  = W_(i)^T W_(i) / N   of the current (updated) block            (two kernels, fixed summation order)
//     T_wush  = Algorithm 1 (M_W(i), M_X(i), lambda), stored as bf16;  T_xvsh = (stored T)^-T, kept as fp32
//     Hbar    = T (L_ii L_ii^T)^-1 T^T;  Lb = lower Cholesky factor of Hbar^-1 = T^-T L_ii L_ii^T T^-1
//     per output channel n (one thread each):  wbar = T_xvsh w_n;  scale from AbsMax(wbar);  for q = 0..d-1:
//         code_q = E2M1(wbar_q / scale);  err = (wbar_q - dequant) / Lb[q][q];  wbar_r -= Lb[r][q] err  (r > q)
//       what_n = T^T dequant  (back in the original space);  E_n = what_n - w_n;  Z_n = L_ii^-1 E_n;  w_n <- what_n
//     W[:, later columns k] += sum_c Z[:, c] * L[k][i*d + c]                  (inter-block propagation)
#include "../../include/wush.h"
#include "wush_device.cuh"
#include "wush_host.h"
#include "wush_linalg.cuh"

namespace wush {
namespace gq {

constexpr int MOM_PARTS = 64;        // CTAs (= partial sums) of the block-moment kernel
constexpr int GROUP = 8;             // blocks whose updates of the far columns are applied in one pass

// ---------------------------------------------------------------------------------------- preparation
__global__ void to_f64_kernel(const __nv_bfloat16* __restrict__ W, double* __restrict__ out, int64_t n) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    out[i] = (double)__bfloat162float(W[i]);
}

// H[a][b] = sum_t X[t][a] X[t][b] / B, 32 x 32 tile per CTA (256 threads, 4 outputs each); tokens in a fixed order
__global__ void __launch_bounds__(256)
hessian_kernel(const __nv_bfloat16* __restrict__ X, int64_t B, int64_t K, double* __restrict__ H) {
  __shared__ double xa[32][33], xb[32][33];
  const int a0 = blockIdx.y * 32, b0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;         // ty 0..7
  double acc[4] = {0.0, 0.0, 0.0, 0.0};
  for (int64_t t0 = 0; t0 < B; t0 += 32) {
    for (int r = ty; r < 32; r += 8) {
      const int64_t t = t0 + r;
      xa[r][tx] = (t < B && a0 + tx < K) ? (double)__bfloat162float(X[t * K + a0 + tx]) : 0.0;
      xb[r][tx] = (t < B && b0 + tx < K) ? (double)__bfloat162float(X[t * K + b0 + tx]) : 0.0;
    }
    __syncthreads();
#pragma unroll 8
    for (int r = 0; r < 32; ++r) {
      const double vb = xb[r][tx];
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[e] += xa[r][ty + 8 * e] * vb;
    }
    __syncthreads();
  }
  const double inv = 1.0 / (double)B;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const int a = a0 + ty + 8 * e, b = b0 + tx;
    if (a < K && b < K) H[(int64_t)a * K + b] = acc[e] * inv;
  }
}

// diagonal blocks of the undamped Hessian -> MX[C][d][d]
__global__ void diag_blocks_kernel(const double* __restrict__ H, int64_t K, int d, double* __restrict__ MX) {
  const int c = blockIdx.x;
  for (int idx = threadIdx.x; idx < d * d; idx += blockDim.x)
    MX[(int64_t)c * d * d + idx] = H[((int64_t)c * d + idx / d) * K + (int64_t)c * d + idx % d];
}

// H += lambda * tr(H)/K * I; the trace is summed by one CTA in a fixed order
__global__ void __launch_bounds__(256) damp_kernel(double* __restrict__ H, int64_t K, double lambda) {
  __shared__ double part[256];
  double s = 0.0;
  for (int64_t i = threadIdx.x; i < K; i += 256) s += H[i * K + i];
  part[threadIdx.x] = s;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
    __syncthreads();
  }
  const double add = lambda * part[0] / (double)K;
  for (int64_t i = threadIdx.x; i < K; i += 256) H[i * K + i] += add;
}

// One column of the factorisation Hd = U U^T (U upper triangular, stored in the upper triangle of A in place),
// columns taken from the last to the first:
//   U[j][j] = sqrt(A[j][j] - sum_{k>j} U[j][k]^2),   U[i][j] = (A[i][j] - sum_{k>j} U[i][k] U[j][k]) / U[j][j], i < j.
// Every CTA recomputes the pivot (same order, same value) and none stores it (see below).  One warp per row i.
__global__ void __launch_bounds__(256) ul_column_kernel(double* __restrict__ A, int64_t K, int j, int* __restrict__ fail) {
  __shared__ double part[256];
  __shared__ double pivot;
  const double* rj = A + (int64_t)j * K;
  double s = 0.0;
  for (int64_t k = j + 1 + threadIdx.x; k < K; k += 256) s += rj[k] * rj[k];
  part[threadIdx.x] = s;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    double p = rj[j] - part[0];
    if (!(p > 0.0)) { if (blockIdx.x == 0) *fail = 1; p = 1.0; }
    pivot = sqrt(p);
  }
  __syncthreads();
  const double piv = pivot;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = blockIdx.x * 8 + warp; i < j; i += gridDim.x * 8) {
    const double* ri = A + (int64_t)i * K;
    double t = 0.0;
    for (int64_t k = j + 1 + lane; k < K; k += 32) t += ri[k] * rj[k];
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (lane == 0) A[(int64_t)i * K + j] = (ri[j] - t) / piv;
  }
}
// U[j][j] itself, stored by a kernel of its own (one CTA, the same sum in the same order) after the column kernel,
// so that the column kernel never writes an element that its other CTAs still read
__global__ void __launch_bounds__(256) ul_store_pivot_kernel(double* __restrict__ A, int64_t K, int j) {
  __shared__ double part[256];
  const double* rj = A + (int64_t)j * K;
  double s = 0.0;
  for (int64_t k = j + 1 + threadIdx.x; k < K; k += 256) s += rj[k] * rj[k];
  part[threadIdx.x] = s;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    double p = rj[j] - part[0];
    if (!(p > 0.0)) p = 1.0;
    A[(int64_t)j * K + j] = sqrt(p);
  }
}

// One row of V = U^-1 (upper triangular), rows taken from the last to the first:
//   V[i][i] = 1 / U[i][i],   V[i][c] = -(sum_{k = i+1..c} U[i][k] V[k][c]) / U[i][i]   for c > i.
// A CTA takes 32 columns (lane = column, so V[k][c] is read along rows); its 16 warps take the terms k = i+1+w,
// i+1+w+16, ... and the 16 partial sums are added in warp order, so the result is the same from run to run.
// (One thread per column walking all of its terms made this kernel nine tenths of the solver's time.)
constexpr int UINV_WARPS = 16;
__global__ void __launch_bounds__(32 * UINV_WARPS) uinv_row_kernel(const double* __restrict__ U, double* __restrict__ V, int64_t K, int i) {
  __shared__ double part[UINV_WARPS][32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int64_t c = (int64_t)i + 1 + (int64_t)blockIdx.x * 32 + lane;
  const double* ui = U + (int64_t)i * K;
  double s = 0.0;
  if (c < K)
    for (int64_t k = (int64_t)i + 1 + w; k <= c; k += UINV_WARPS) s += ui[k] * V[k * K + c];
  part[w][lane] = s;
  __syncthreads();
  const double inv = 1.0 / ui[i];
  if (w == 0 && c < K) {
    double t = 0.0;
#pragma unroll
    for (int q = 0; q < UINV_WARPS; ++q) t += part[q][lane];
    V[(int64_t)i * K + c] = -t * inv;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) V[(int64_t)i * K + i] = inv;
}
__global__ void zero_lower_kernel(double* __restrict__ V, int64_t K) {       // strictly lower part of V := 0
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < K * K; idx += (int64_t)gridDim.x * blockDim.x)
    if (idx % K < idx / K) V[idx] = 0.0;
}

// ---------------------------------------------------------------------------------------- per block
// Partial second-moment sums of the current block: part p adds rows p, p + MOM_PARTS, ... in that order.
template <int D>
__global__ void __launch_bounds__(256)
block_moment_partial_kernel(const double* __restrict__ Wc, int64_t N, int64_t K, int blk, double* __restrict__ partial) {
  __shared__ double row[D];
  constexpr int PER = D * D / 256;                     // 4 (D = 32) or 1 (D = 16)
  double acc[PER];
#pragma unroll
  for (int e = 0; e < PER; ++e) acc[e] = 0.0;
  for (int64_t n = blockIdx.x; n < N; n += MOM_PARTS) {
    if (threadIdx.x < D) row[threadIdx.x] = Wc[n * K + (int64_t)blk * D + threadIdx.x];
    __syncthreads();
#pragma unroll
    for (int e = 0; e < PER; ++e) {
      const int idx = threadIdx.x + 256 * e;
      acc[e] += row[idx / D] * row[idx % D];
    }
    __syncthreads();
  }
#pragma unroll
  for (int e = 0; e < PER; ++e) partial[(int64_t)blockIdx.x * D * D + threadIdx.x + 256 * e] = acc[e];
}
template <int D>
__global__ void __launch_bounds__(256) block_moment_reduce_kernel(const double* __restrict__ partial, double* __restrict__ mw) {
  for (int idx = threadIdx.x; idx < D * D; idx += 256) {
    double s = 0.0;
    for (int p = 0; p < MOM_PARTS; ++p) s += partial[(int64_t)p * D * D + idx];
    mw[idx] = s;
  }
}

// Lb = lower Cholesky factor of Hbar^-1 = Tx L_ii L_ii^T Tx^T, Tx = (stored T)^-T in fp64; also L_ii itself, copied
// out of V (L_ii[a][b] = V[i*d + b][i*d + a]).  One CTA.  lmat: [0 .. d*d) = Lb, [d*d .. 2 d*d) = L_ii.
template <int D>
__global__ void __launch_bounds__(BT_THREADS)
block_hessian_kernel(const __nv_bfloat16* __restrict__ T, const double* __restrict__ V, int64_t K, int blk,
                     double* __restrict__ lmat, float* __restrict__ tinv_scratch, int32_t* __restrict__ info) {
  __shared__ double Tm[D * D], Rm[D * D], Lii[D * D], Gm[D * D];
  __shared__ double fac[D];
  __shared__ int perm[D];
  __shared__ int fail;
  const int tid = threadIdx.x;
  if (tid == 0) fail = 0;
  for (int idx = tid; idx < D * D; idx += BT_THREADS) {
    const int a = idx / D, b = idx % D;
    Tm[idx] = (double)__bfloat162float(T[idx]);
    Lii[idx] = (b <= a) ? V[((int64_t)blk * D + b) * K + (int64_t)blk * D + a] : 0.0;
  }
  __syncthreads();
  inverse_transpose<D>(Tm, Rm, fac, perm, &fail, tinv_scratch);        // Rm = T^-1, so Tx[a][k] = Rm[k][a]
  __syncthreads();
  for (int idx = tid; idx < D * D; idx += BT_THREADS) {                // G = Tx L_ii
    const int a = idx / D, b = idx % D;
    double s = 0.0;
    for (int k = b; k < D; ++k) s += Rm[k * D + a] * Lii[k * D + b];
    Gm[idx] = s;
  }
  __syncthreads();
  for (int idx = tid; idx < D * D; idx += BT_THREADS) {                // Hbar^-1 = G G^T (into Tm)
    const int a = idx / D, b = idx % D;
    double s = 0.0;
    for (int k = 0; k < D; ++k) s += Gm[a * D + k] * Gm[b * D + k];
    Tm[idx] = s;
  }
  __syncthreads();
  cholesky_lower<D>(Tm, &fail);
  for (int idx = tid; idx < D * D; idx += BT_THREADS) { lmat[idx] = Tm[idx]; lmat[D * D + idx] = Lii[idx]; }
  __syncthreads();
  if (tid == 0 && fail != 0 && info != nullptr && info[blk] == 0) info[blk] = fail == 1 ? 4 : fail;
}

// The GPTQ subroutine on the transformed block plus the block's error in the original space: one thread per output
// channel n.  FMT: kFmtMX / kFmtNV.  tmat: the stored transform (bf16) and its fp32 inverse-transpose for this block;
// lmat as written by block_hessian_kernel.  Writes the channel's d codes and its scale byte, replaces the block of
// Wc by its dequantised value in the original space and leaves Z_n = L_ii^-1 (what_n - w_n) in Z[n][0..d).
template <int D, int FMT>
__global__ void __launch_bounds__(128)
block_quant_kernel(double* __restrict__ Wc, int64_t N, int64_t K, int blk, const __nv_bfloat16* __restrict__ T,
                   const float* __restrict__ Tinv, const double* __restrict__ lmat, const float* __restrict__ ts_ptr,
                   int mx_ceil, uint8_t* __restrict__ codes, uint8_t* __restrict__ scales, int sf_layout, int64_t KB,
                   double* __restrict__ Z) {
  __shared__ double Ts[D * D], Tx[D * D], Lb[D * D], Lii[D * D];
  for (int idx = threadIdx.x; idx < D * D; idx += 128) {
    Ts[idx] = (double)__bfloat162float(T[idx]);
    Tx[idx] = (double)Tinv[idx];
    Lb[idx] = lmat[idx];
    Lii[idx] = lmat[D * D + idx];
  }
  __syncthreads();
  const int64_t n = (int64_t)blockIdx.x * 128 + threadIdx.x;
  if (n >= N) return;
  double* wrow = Wc + n * K + (int64_t)blk * D;
  double wb[D];                                        // transformed block, then its dequantised values
#pragma unroll
  for (int q = 0; q < D; ++q) wb[q] = 0.0;
  for (int k = 0; k < D; ++k) {                        // wbar = T_xvsh w
    const double wk = wrow[k];
#pragma unroll
    for (int q = 0; q < D; ++q) wb[q] += Tx[q * D + k] * wk;
  }
  float amax = 0.0f;
#pragma unroll
  for (int q = 0; q < D; ++q) amax = fmaxf(amax, fabsf((float)wb[q]));
  uint32_t sbyte;
  float mult;
  double dq;
  if (FMT == kFmtMX) {
    mx_scale(amax, sbyte, mult, mx_ceil);
    dq = 1.0 / (double)mult;                           // 2^e, exact
  } else {
    const float ts = *ts_ptr;
    nv_scale(amax, ts, sbyte, mult);
    dq = (double)e4m3_to_float(sbyte) * (double)ts;    // what a code stands for: no fp32 rounding of the product
  }
  uint32_t packed[D / 8];
#pragma unroll
  for (int w = 0; w < D / 8; ++w) packed[w] = 0;
#pragma unroll
  for (int q = 0; q < D; ++q) {
    const float u = __fmul_rn((float)wb[q], mult);
    const uint32_t code = (uint32_t)__nv_cvt_float2_to_fp4x2(make_float2(u, 0.0f), __NV_E2M1, cudaRoundNearest) & 0xFu;
    packed[q / 8] |= code << (4 * (q % 8));
    const uint32_t mag = code & 7u;
    const double gv = (mag < 4u) ? 0.5 * (double)mag : (mag == 4u ? 2.0 : (mag == 5u ? 3.0 : (mag == 6u ? 4.0 : 6.0)));
    const double deq = __dmul_rn((code & 8u) ? -gv : gv, dq);
    const double err = __ddiv_rn(__dsub_rn(wb[q], deq), Lb[q * D + q]);
#pragma unroll
    for (int r = q + 1; r < D; ++r) wb[r] = __dsub_rn(wb[r], __dmul_rn(Lb[r * D + q], err));
    wb[q] = deq;
  }
  uint8_t* cdst = codes + n * (K >> 1) + (int64_t)blk * (D / 2);
#pragma unroll
  for (int w = 0; w < D / 8; ++w) reinterpret_cast<uint32_t*>(cdst)[w] = packed[w];
  scales[sf_offset(sf_layout, n, blk, KB)] = (uint8_t)sbyte;
  // back to the original space: what = T^T dequant (T_xvsh^-1 = T_wush^T, Eq. 6); E = what - w; Z = L_ii^-1 E
  double z[D];
  for (int k = 0; k < D; ++k) {
    double s = 0.0;
#pragma unroll
    for (int q = 0; q < D; ++q) s += Ts[q * D + k] * wb[q];
    const double e = s - wrow[k];
    wrow[k] = s;
    z[k] = e;
  }
#pragma unroll
  for (int a = 0; a < D; ++a) {
    double s = z[a];
#pragma unroll
    for (int b = 0; b < a; ++b) s -= Lii[a * D + b] * z[b];
    z[a] = s / Lii[a * D + a];
  }
  double* zrow = Z + n * D;
#pragma unroll
  for (int a = 0; a < D; ++a) zrow[a] = z[a];
}

// Inter-block propagation for columns k in [k_begin, k_end) and the nb blocks blk0 .. blk0 + nb - 1 whose Z is stored
// (Z of block blk0 + t at Z + t * N * D):
//   Wc[n][k] <- (..((Wc[n][k] + u_0) + u_1).. + u_{nb-1}),   u_t = sum_c Z_t[n][c] * L[k][(blk0 + t)*d + c],  L[k][j] = V[j][k]
// - the additions in block order, each u_t summed over c in order, exactly as if every block had updated all later
// columns right away.  The solver uses it twice: with nb = 1 for the columns of the current group of blocks (the next
// block needs them at once) and with nb = the group size for everything beyond the group (one pass over the far
// columns per group instead of one per block).  A thread owns one column and walks 32 rows.
template <int D>
__global__ void __launch_bounds__(256)
propagate_kernel(double* __restrict__ Wc, int64_t N, int64_t K, int blk0, int nb, int64_t k_begin, int64_t k_end,
                 const double* __restrict__ V, const double* __restrict__ Z) {
  __shared__ double zs[32][D];
  const int64_t k = k_begin + (int64_t)blockIdx.x * 256 + threadIdx.x;
  const int64_t n0 = (int64_t)blockIdx.y * 32;
  const bool live = k < k_end;
  double w[32];
#pragma unroll
  for (int r = 0; r < 32; ++r) w[r] = (live && n0 + r < N) ? Wc[(n0 + r) * K + k] : 0.0;
  for (int t = 0; t < nb; ++t) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < 32 * D; idx += 256) {
      const int64_t n = n0 + idx / D;
      zs[idx / D][idx % D] = (n < N) ? Z[((int64_t)t * N + n) * D + idx % D] : 0.0;
    }
    __syncthreads();
    if (!live) continue;
    double v[D];
#pragma unroll
    for (int c = 0; c < D; ++c) v[c] = V[((int64_t)(blk0 + t) * D + c) * K + k];
#pragma unroll
    for (int r = 0; r < 32; ++r) {
      double s = 0.0;
#pragma unroll
      for (int c = 0; c < D; ++c) s += zs[r][c] * v[c];
      w[r] += s;
    }
  }
  if (!live) return;
#pragma unroll
  for (int r = 0; r < 32; ++r)
    if (n0 + r < N) Wc[(n0 + r) * K + k] = w[r];
}

// a failed factorisation of the damped Hessian (non-positive pivot) is reported on every block
__global__ void report_failure_kernel(const int* __restrict__ fail, int32_t* __restrict__ info, int C) {
  if (*fail == 0) return;
  for (int c = threadIdx.x; c < C; c += blockDim.x) if (info[c] == 0) info[c] = 5;
}

}  // namespace gq

// ---------------------------------------------------------------------------------------- host side
// workspace: Wc [N][K] | A (Hd, then U) [K][K] | V [K][K] | MX [K/d][d][d] | Z [N][d] | partial [MOM_PARTS][d][d] |
//            mw [d][d] | lmat [2][d][d] | fail flag          (Z holds the last GROUP blocks' [N][d])
static inline size_t up256(size_t x) { return (x + 255) & ~size_t(255); }
size_t gptq_workspace_bytes(int64_t N, int64_t K, int g) {
  const size_t d2 = (size_t)g * g * sizeof(double);
  return up256((size_t)N * K * 8) + 2 * up256((size_t)K * K * 8) + up256((size_t)K * g * 8) + up256((size_t)gq::GROUP * N * g * 8) +
         up256(gq::MOM_PARTS * d2) + up256(d2) + up256(2 * d2) + 256;
}

template <int D>
static cudaError_t gptq_run(const void* W, int64_t N, int64_t K, const void* Xc, int64_t B, int fmt, double lambda,
                            const float* ts_w, void* T, float* Tinv, uint8_t* codes, uint8_t* scales, int sf,
                            int32_t* info, void* workspace, int mx_ceil, cudaStream_t st) {
  using namespace gq;
  const int C = (int)(K / D);
  const size_t d2 = (size_t)D * D * sizeof(double);
  uint8_t* p = reinterpret_cast<uint8_t*>(workspace);
  double* Wc = reinterpret_cast<double*>(p); p += up256((size_t)N * K * 8);
  double* A = reinterpret_cast<double*>(p); p += up256((size_t)K * K * 8);
  double* V = reinterpret_cast<double*>(p); p += up256((size_t)K * K * 8);
  double* MX = reinterpret_cast<double*>(p); p += up256((size_t)K * D * 8);
  double* Z = reinterpret_cast<double*>(p); p += up256((size_t)GROUP * N * D * 8);
  double* partial = reinterpret_cast<double*>(p); p += up256(MOM_PARTS * d2);
  double* mw = reinterpret_cast<double*>(p); p += up256(d2);
  double* lmat = reinterpret_cast<double*>(p); p += up256(2 * d2);
  int* fail = reinterpret_cast<int*>(p);
  cudaError_t e;
#define GQ_CHECK() do { if ((e = cudaGetLastError()) != cudaSuccess) return e; } while (0)
  if ((e = cudaMemsetAsync(fail, 0, sizeof(int), st)) != cudaSuccess) return e;
  if (info != nullptr && (e = cudaMemsetAsync(info, 0, sizeof(int32_t) * C, st)) != cudaSuccess) return e;
  to_f64_kernel<<<1184, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(W), Wc, N * K); GQ_CHECK();
  const unsigned kt = (unsigned)((K + 31) / 32);
  hessian_kernel<<<dim3(kt, kt), 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(Xc), B, K, A); GQ_CHECK();
  diag_blocks_kernel<<<C, 256, 0, st>>>(A, K, D, MX); GQ_CHECK();
  damp_kernel<<<1, 256, 0, st>>>(A, K, lambda); GQ_CHECK();
  for (int j = (int)K - 1; j >= 0; --j) {                 // Hd = U U^T, last column first
    if (j > 0) {
      const int grid = (j + 7) / 8 < 592 ? (j + 7) / 8 : 592;
      ul_column_kernel<<<grid, 256, 0, st>>>(A, K, j, fail); GQ_CHECK();
    }
    ul_store_pivot_kernel<<<1, 256, 0, st>>>(A, K, j); GQ_CHECK();
  }
  zero_lower_kernel<<<1184, 256, 0, st>>>(V, K); GQ_CHECK();
  for (int i = (int)K - 1; i >= 0; --i) {                 // V = U^-1, last row first
    uinv_row_kernel<<<(unsigned)((K - i - 1 + 31) / 32 > 0 ? (K - i - 1 + 31) / 32 : 1), 32 * UINV_WARPS, 0, st>>>(A, V, K, i); GQ_CHECK();
  }
  __nv_bfloat16* Tb = reinterpret_cast<__nv_bfloat16*>(T);
  for (int i = 0; i < C; ++i) {
    block_moment_partial_kernel<D><<<MOM_PARTS, 256, 0, st>>>(Wc, N, K, i, partial); GQ_CHECK();
    block_moment_reduce_kernel<D><<<1, 256, 0, st>>>(partial, mw); GQ_CHECK();
    // Algorithm 1 on (M_W of the updated block, M_X = diagonal block of the Hessian, already divided by B)
    if ((e = run_build_transform_f64(mw, 1.0 / (double)N, MX + (size_t)i * D * D, 1.0, D, lambda, Tb + (size_t)i * D * D,
                                     Tinv + (size_t)i * D * D, info ? info + i : nullptr, st)) != cudaSuccess) return e;
    block_hessian_kernel<D><<<1, BT_THREADS, 0, st>>>(Tb + (size_t)i * D * D, V, K, i, lmat, Tinv + (size_t)i * D * D, info); GQ_CHECK();
    const unsigned qgrid = (unsigned)((N + 127) / 128);
    const int t = i % GROUP;                                  // position inside the current group of blocks
    double* Zi = Z + (size_t)t * N * D;
    if (fmt == kFmtMX)
      block_quant_kernel<D, kFmtMX><<<qgrid, 128, 0, st>>>(Wc, N, K, i, Tb + (size_t)i * D * D, Tinv + (size_t)i * D * D, lmat, ts_w,
                                                          mx_ceil, codes, scales, sf, K / D, Zi);
    else
      block_quant_kernel<D, kFmtNV><<<qgrid, 128, 0, st>>>(Wc, N, K, i, Tb + (size_t)i * D * D, Tinv + (size_t)i * D * D, lmat, ts_w,
                                                          0, codes, scales, sf, K / D, Zi);
    GQ_CHECK();
    // this block's update: at once for the rest of its group, together with the group's other blocks for all columns
    // beyond the group (same additions in the same order either way)
    const int group_first = i - t;
    const int64_t group_end = (int64_t)min(group_first + GROUP, C) * D;
    const int64_t near_begin = (int64_t)(i + 1) * D;
    const unsigned ny = (unsigned)((N + 31) / 32);
    if (near_begin < group_end) {
      propagate_kernel<D><<<dim3((unsigned)((group_end - near_begin + 255) / 256), ny), 256, 0, st>>>(Wc, N, K, i, 1, near_begin, group_end, V, Zi);
      GQ_CHECK();
    }
    if ((t == GROUP - 1 || i == C - 1) && group_end < K) {
      propagate_kernel<D><<<dim3((unsigned)((K - group_end + 255) / 256), ny), 256, 0, st>>>(Wc, N, K, group_first, t + 1, group_end, K, V, Z);
      GQ_CHECK();
    }
  }
  if (info != nullptr) { report_failure_kernel<<<1, 256, 0, st>>>(fail, info, C); GQ_CHECK(); }
#undef GQ_CHECK
  return cudaSuccess;
}

cudaError_t run_gptq_quantize_weight(const void* W, int64_t N, int64_t K, const void* Xc, int64_t B, int fmt, int g,
                                     double lambda, const float* ts_w, void* T, float* Tinv, uint8_t* codes,
                                     uint8_t* scales, int sf, int32_t* info, void* workspace, int mx_ceil, cudaStream_t st) {
  if (g == 32) return gptq_run<32>(W, N, K, Xc, B, fmt, lambda, ts_w, T, Tinv, codes, scales, sf, info, workspace, mx_ceil, st);
  return gptq_run<16>(W, N, K, Xc, B, fmt, lambda, ts_w, T, Tinv, codes, scales, sf, info, workspace, mx_ceil, st);
}

}  // namespace wush
