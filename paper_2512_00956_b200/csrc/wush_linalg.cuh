// Small dense fp64 routines that run inside one CTA of BT_THREADS threads on d x d matrices in shared memory
// (d = 16 or 32): in-place lower Cholesky and Gauss-Jordan inverse.  Shared by the transform builder
// (Algorithm 1) and the GPTQ solver (Algorithm 2, GPTQ case).
#pragma once
#include <stdint.h>

namespace wush {

constexpr int BT_THREADS = 128;

template <int D>
__device__ void cholesky_lower(double* A, int* fail) {       // in place; upper triangle zeroed
  for (int j = 0; j < D; ++j) {
    __syncthreads();
    if (threadIdx.x == 0) {
      double s = A[j * D + j];
      for (int k = 0; k < j; ++k) s -= A[j * D + k] * A[j * D + k];
      if (!(s > 0.0)) { *fail = 1; s = 1.0; }
      A[j * D + j] = sqrt(s);
    }
    __syncthreads();
    const double piv = A[j * D + j];
    for (int i = j + 1 + threadIdx.x; i < D; i += BT_THREADS) {
      double s = A[i * D + j];
      for (int k = 0; k < j; ++k) s -= A[i * D + k] * A[j * D + k];
      A[i * D + j] = s / piv;
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < D * D; idx += BT_THREADS)
    if ((idx % D) > (idx / D)) A[idx] = 0.0;
  __syncthreads();
}

// Gauss-Jordan with partial pivoting on the D x D matrix Tm (destroyed); Rm becomes the inverse, fac holds D
// scratch values; the TRANSPOSE of the inverse is written to out (fp32).  *fail = 3 if a pivot is zero.
template <int D>
__device__ void inverse_transpose(double* Tm, double* Rm, double* fac_buf, int* perm, int* fail_ptr, float* out) {
  const int tid = threadIdx.x;
  for (int idx = tid; idx < D * D; idx += BT_THREADS) Rm[idx] = ((idx / D) == (idx % D)) ? 1.0 : 0.0;
  __syncthreads();
  for (int col = 0; col < D; ++col) {
    if (tid == 0) {
      int pr = col; double pv = fabs(Tm[col * D + col]);
      for (int r = col + 1; r < D; ++r) if (fabs(Tm[r * D + col]) > pv) { pv = fabs(Tm[r * D + col]); pr = r; }
      perm[0] = pr;
      if (!(pv > 0.0)) *fail_ptr = 3;
    }
    __syncthreads();
    const int pr = perm[0];
    if (pr != col) {
      for (int k = tid; k < D; k += BT_THREADS) {
        double t = Tm[col * D + k]; Tm[col * D + k] = Tm[pr * D + k]; Tm[pr * D + k] = t;
        t = Rm[col * D + k]; Rm[col * D + k] = Rm[pr * D + k]; Rm[pr * D + k] = t;
      }
    }
    __syncthreads();
    const double piv = Tm[col * D + col];
    __syncthreads();
    for (int k = tid; k < D; k += BT_THREADS) { Tm[col * D + k] /= piv; Rm[col * D + k] /= piv; }
    __syncthreads();
    // eliminate column `col` from every other row; factors are read before any row is modified
    {
      double* fac = fac_buf;
      for (int r = tid; r < D; r += BT_THREADS) fac[r] = (r == col) ? 0.0 : Tm[r * D + col];
      __syncthreads();
      for (int idx = tid; idx < D * D; idx += BT_THREADS) {
        const int r = idx / D, k = idx % D;
        const double f = fac[r];
        if (f != 0.0) { Tm[idx] -= f * Tm[col * D + k]; Rm[idx] -= f * Rm[col * D + k]; }
      }
    }
    __syncthreads();
  }
  for (int idx = tid; idx < D * D; idx += BT_THREADS) {
    const int j = idx / D, k = idx % D;
    out[idx] = (float)Rm[k * D + j];      // transpose of the inverse
  }
}

}  // namespace wush
