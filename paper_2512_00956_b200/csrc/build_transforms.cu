// Algorithm 1 ("Compute WUSH for One Block") and the inverse-transpose pairing of Eq. 6 on the
// device: one CTA per block of d = g channels, everything in fp64 in shared memory.
//
//   M_W, M_X   <- moment sums / row counts, symmetrised, damped:  M + lambda * tr(M)/d * I
//   W', X'     <- lower Cholesky factors
//   U S V^T    <- SVD of W'^T X', by one-sided Jacobi on (W'^T X')^T = X'^T W' (its right singular
//                 vectors are U); round-robin pair ordering, d/2 independent rotations per step
//   T_wush     <- H S^-1/2 U^T W'^T   (singular values descending; each row of U^T W'^T signed so that its
//                 largest-magnitude entry is positive - Lemma A.1's factor-independent quantity)
//   T_hat      <- bf16(T_wush)                      (what the online kernel multiplies activations with)
//   T_xvsh     <- (T_hat)^-T in fp64, stored as fp32 (what the offline weight path uses)
//
// This is offline glue between the calibration-moment kernel and the weight quantiser: O(d^3) per
// block, a few hundred blocks per layer.  info[c] != 0 flags a block whose factorisation failed
// (1: non-positive Cholesky pivot, 2: Jacobi did not converge, 3: singular transform).
#include "../../include/wush.h"
#include "wush_device.cuh"
#include "wush_host.h"
#include "wush_linalg.cuh"

namespace wush {

template <int D, typename MT = float>
__global__ void __launch_bounds__(BT_THREADS)
build_transforms_kernel(const MT* __restrict__ mom_w, double inv_nw, const MT* __restrict__ mom_x, double inv_nx,
                        double lambda, __nv_bfloat16* __restrict__ T_out, float* __restrict__ Tinv_out,
                        int32_t* __restrict__ info, int with_hadamard) {
  extern __shared__ double sm[];
  double* Wp = sm;                 // M_W -> W'
  double* Xp = Wp + D * D;         // M_X -> X'
  double* Bm = Xp + D * D;         // X'^T W', columns orthogonalised by Jacobi
  double* Jm = Bm + D * D;         // accumulated rotations = U
  double* Rm = Jm + D * D;         // U^T W'^T (sorted, signed), later the inverse work matrix
  double* Tm = Rm + D * D;         // T_wush / T_hat
  __shared__ double sigma[D];
  __shared__ double red[2];
  __shared__ int perm[D];
  __shared__ int fail, rotated;
  const int c = blockIdx.x, tid = threadIdx.x;
  const MT* mw = mom_w + (size_t)c * D * D;
  const MT* mx = mom_x + (size_t)c * D * D;
  if (tid == 0) { fail = 0; red[0] = red[1] = 0.0; }
  __syncthreads();

  // ---- moments: normalise, symmetrise, damp
  for (int idx = tid; idx < D * D; idx += BT_THREADS) {
    const int i = idx / D, j = idx % D;
    Wp[idx] = 0.5 * ((double)mw[i * D + j] + (double)mw[j * D + i]) * inv_nw;
    Xp[idx] = 0.5 * ((double)mx[i * D + j] + (double)mx[j * D + i]) * inv_nx;
  }
  __syncthreads();
  if (tid == 0) {
    double tw = 0.0, tx = 0.0;
    for (int i = 0; i < D; ++i) { tw += Wp[i * D + i]; tx += Xp[i * D + i]; }
    red[0] = lambda * tw / D; red[1] = lambda * tx / D;
  }
  __syncthreads();
  if (tid < D) { Wp[tid * D + tid] += red[0]; Xp[tid * D + tid] += red[1]; }
  __syncthreads();
  cholesky_lower<D>(Wp, &fail);
  cholesky_lower<D>(Xp, &fail);

  // ---- B = X'^T W'  (= (W'^T X')^T),  J = I
  for (int idx = tid; idx < D * D; idx += BT_THREADS) {
    const int i = idx / D, j = idx % D;
    double s = 0.0;
    for (int k = 0; k < D; ++k) s += Xp[k * D + i] * Wp[k * D + j];
    Bm[idx] = s;
    Jm[idx] = (i == j) ? 1.0 : 0.0;
  }
  __syncthreads();

  // ---- one-sided Jacobi: rotate column pairs of B (and J) until all pairs are orthogonal.
  // Round-robin schedule: D-1 steps per sweep, D/2 disjoint pairs per step; a group of GS threads owns a pair.
  constexpr int PAIRS = D / 2;
  constexpr int GS = BT_THREADS / PAIRS;            // 8 (D = 32) or 16 (D = 16) threads per pair
  const int pair = tid / GS, gl = tid % GS;
  const unsigned gmask = (GS == 32) ? 0xffffffffu : (((1u << GS) - 1u) << ((tid % 32) / GS * GS));
  int sweep = 0;
  for (; sweep < 40; ++sweep) {
    if (tid == 0) rotated = 0;
    __syncthreads();
    for (int step = 0; step < D - 1; ++step) {
      // circle method: index 0 stays, indices 1..D-1 rotate; slot m meets slot D-1-m
      const int a = (pair == 0) ? 0 : (pair + step) % (D - 1) + 1;
      const int b = (pair == 0) ? step % (D - 1) + 1 : (D - 1 - pair + step) % (D - 1) + 1;
      const int p = min(a, b), q = max(a, b);
      double al = 0.0, be = 0.0, ga = 0.0;
      for (int r = gl; r < D; r += GS) {
        const double x = Bm[r * D + p], y = Bm[r * D + q];
        al += x * x; be += y * y; ga += x * y;
      }
#pragma unroll
      for (int o = GS / 2; o > 0; o >>= 1) {
        al += __shfl_xor_sync(gmask, al, o);
        be += __shfl_xor_sync(gmask, be, o);
        ga += __shfl_xor_sync(gmask, ga, o);
      }
      if (fabs(ga) > 1e-15 * sqrt(al * be) && al > 0.0 && be > 0.0) {
        const double zeta = (be - al) / (2.0 * ga);
        const double t = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
        const double cs = 1.0 / sqrt(1.0 + t * t), sn = cs * t;
        for (int r = gl; r < D; r += GS) {
          const double x = Bm[r * D + p], y = Bm[r * D + q];
          Bm[r * D + p] = cs * x - sn * y; Bm[r * D + q] = sn * x + cs * y;
          const double u = Jm[r * D + p], v = Jm[r * D + q];
          Jm[r * D + p] = cs * u - sn * v; Jm[r * D + q] = sn * u + cs * v;
        }
        // another sweep while any pair is further from orthogonal than a few rounding errors of its inner product:
        // the transform's entries inherit this residue divided by the relative gap of neighbouring singular values
        if (gl == 0 && fabs(ga) > 1e-14 * sqrt(al * be)) rotated = 1;
      }
      __syncthreads();
    }
    if (rotated == 0) break;
    __syncthreads();
  }
  if (tid == 0 && sweep >= 40) fail = 2;

  // ---- singular values, descending order
  if (tid < D) {
    double s = 0.0;
    for (int r = 0; r < D; ++r) s += Bm[r * D + tid] * Bm[r * D + tid];
    sigma[tid] = sqrt(s);
  }
  __syncthreads();
  if (tid < D) {
    int rank = 0;
    for (int j = 0; j < D; ++j) rank += (sigma[j] > sigma[tid]) || (sigma[j] == sigma[tid] && j < tid);
    perm[rank] = tid;
  }
  __syncthreads();

  // ---- R = U^T W'^T, rows in sorted order, signed
  for (int idx = tid; idx < D * D; idx += BT_THREADS) {
    const int i = idx / D, k = idx % D;
    const int ci = perm[i];
    double s = 0.0;
    for (int m = 0; m < D; ++m) s += Jm[m * D + ci] * Wp[k * D + m];
    Rm[idx] = s;
  }
  __syncthreads();
  if (tid < D) {
    int best = 0; double bv = -1.0;
    for (int k = 0; k < D; ++k) { const double v = fabs(Rm[tid * D + k]); if (v > bv) { bv = v; best = k; } }
    const double sg = (Rm[tid * D + best] < 0.0) ? -1.0 : 1.0;
    const double sc = sg / sqrt(sigma[perm[tid]]);
    for (int k = 0; k < D; ++k) Rm[tid * D + k] *= sc;              // S^-1/2 folded in
  }
  __syncthreads();

  // ---- T = H (S^-1/2 R),  H[a][i] = (-1)^popcount(a & i) / sqrt(D);  T_hat = bf16(T)
  const double hnorm = rsqrt((double)D);
  for (int idx = tid; idx < D * D; idx += BT_THREADS) {
    const int a = idx / D, k = idx % D;
    double s = 0.0;
    if (with_hadamard) {
      for (int i = 0; i < D; ++i) s += ((__popc(a & i) & 1) ? -Rm[i * D + k] : Rm[i * D + k]);
      s *= hnorm;
    } else {
      s = Rm[idx];                                   // "WUS": the same transform without the Hadamard factor
    }
    const __nv_bfloat16 tb = __double2bfloat16(s);
    T_out[(size_t)c * D * D + idx] = tb;
    Tm[idx] = (double)__bfloat162float(tb);
  }
  __syncthreads();

  inverse_transpose<D>(Tm, Rm, Bm, perm, &fail, Tinv_out + (size_t)c * D * D);
  if (tid == 0 && info != nullptr) info[c] = fail;
}

// (T)^-T of given bf16 transforms (Eq. 6 for transforms that were not built here)
template <int D>
__global__ void __launch_bounds__(BT_THREADS)
invert_transforms_kernel(const __nv_bfloat16* __restrict__ T, float* __restrict__ Tinv_out, int32_t* __restrict__ info) {
  extern __shared__ double sm[];
  double* Tm = sm;
  double* Rm = Tm + D * D;
  double* fac = Rm + D * D;
  __shared__ int perm[D];
  __shared__ int fail;
  const int c = blockIdx.x, tid = threadIdx.x;
  if (tid == 0) fail = 0;
  for (int idx = tid; idx < D * D; idx += BT_THREADS) Tm[idx] = (double)__bfloat162float(T[(size_t)c * D * D + idx]);
  __syncthreads();
  inverse_transpose<D>(Tm, Rm, fac, perm, &fail, Tinv_out + (size_t)c * D * D);
  __syncthreads();
  if (tid == 0 && info != nullptr) info[c] = fail;
}

cudaError_t run_invert_transforms(const void* T, int64_t K, int g, float* Tinv, int32_t* info, cudaStream_t st) {
  const int C = (int)(K / g);
  const size_t smem = (2 * (size_t)g * g + g) * sizeof(double);          // <= 16.6 KB: no attribute needed
  const __nv_bfloat16* Tb = reinterpret_cast<const __nv_bfloat16*>(T);
  if (g == 32) invert_transforms_kernel<32><<<C, BT_THREADS, smem, st>>>(Tb, Tinv, info);
  else invert_transforms_kernel<16><<<C, BT_THREADS, smem, st>>>(Tb, Tinv, info);
  return cudaGetLastError();
}

// The data-independent comparison transforms of Sec. 5 / Table 1 written in the layout the kernels take: the
// same normalised Sylvester-Hadamard matrix (kind 0; entries +-d^-1/2 rounded to bf16) or the identity (kind 1)
// for every block.
template <int D>
__global__ void __launch_bounds__(BT_THREADS)
fixed_transforms_kernel(__nv_bfloat16* __restrict__ T, int kind) {
  const float h = rsqrtf((float)D);                      // exact for D = 16, one rounding for D = 32; bf16 below
  for (int idx = threadIdx.x; idx < D * D; idx += BT_THREADS) {
    const int j = idx / D, k = idx % D;
    float v;
    if (kind == 0) v = (__popc(j & k) & 1) ? -h : h;
    else v = (j == k) ? 1.0f : 0.0f;
    T[(size_t)blockIdx.x * D * D + idx] = __float2bfloat16_rn(v);
  }
}

cudaError_t run_fixed_transforms(int kind, int64_t K, int g, void* T, float* Tinv, int32_t* info, cudaStream_t st) {
  const int C = (int)(K / g);
  __nv_bfloat16* Tb = reinterpret_cast<__nv_bfloat16*>(T);
  if (g == 32) fixed_transforms_kernel<32><<<C, BT_THREADS, 0, st>>>(Tb, kind);
  else fixed_transforms_kernel<16><<<C, BT_THREADS, 0, st>>>(Tb, kind);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  return run_invert_transforms(T, K, g, Tinv, info, st);   // Eq. 6 for the stored values
}

cudaError_t run_build_transforms(const float* mom_w, int64_t n_w, const float* mom_x, int64_t n_x, int64_t K, int g,
                                 double lambda, void* T, float* Tinv, int32_t* info, cudaStream_t st, bool with_hadamard) {
  const int wh = with_hadamard ? 1 : 0;
  const int C = (int)(K / g);
  const size_t smem = 6 * (size_t)g * g * sizeof(double);
  __nv_bfloat16* Tb = reinterpret_cast<__nv_bfloat16*>(T);
  cudaError_t e;
  if (g == 32) {
    static bool done_of[kDeviceSlots] = {};              // the attribute belongs to the device's copy of the kernel
    const int slot = device_slot();
    if (slot < 0) return cudaErrorInvalidDevice;
    if (!done_of[slot]) {
      e = cudaFuncSetAttribute(build_transforms_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      done_of[slot] = true;
    }
    build_transforms_kernel<32><<<C, BT_THREADS, smem, st>>>(mom_w, 1.0 / (double)n_w, mom_x, 1.0 / (double)n_x, lambda, Tb, Tinv, info, wh);
  } else {
    build_transforms_kernel<16><<<C, BT_THREADS, smem, st>>>(mom_w, 1.0 / (double)n_w, mom_x, 1.0 / (double)n_x, lambda, Tb, Tinv, info, wh);
  }
  return cudaGetLastError();
}

// One block from fp64 moment sums (the GPTQ case of Algorithm 2 builds its transforms one at a time from the
// updated weights): same kernel, double-precision inputs.
cudaError_t run_build_transform_f64(const double* mom_w, double inv_nw, const double* mom_x, double inv_nx, int g,
                                    double lambda, void* T, float* Tinv, int32_t* info, cudaStream_t st) {
  const size_t smem = 6 * (size_t)g * g * sizeof(double);
  __nv_bfloat16* Tb = reinterpret_cast<__nv_bfloat16*>(T);
  if (g == 32) {
    static bool done_of[kDeviceSlots] = {};
    const int slot = device_slot();
    if (slot < 0) return cudaErrorInvalidDevice;
    if (!done_of[slot]) {
      const cudaError_t e = cudaFuncSetAttribute(build_transforms_kernel<32, double>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      done_of[slot] = true;
    }
    build_transforms_kernel<32, double><<<1, BT_THREADS, smem, st>>>(mom_w, inv_nw, mom_x, inv_nx, lambda, Tb, Tinv, info, 1);
  } else {
    build_transforms_kernel<16, double><<<1, BT_THREADS, smem, st>>>(mom_w, inv_nw, mom_x, inv_nx, lambda, Tb, Tinv, info, 1);
  }
  return cudaGetLastError();
}

}  // namespace wush
