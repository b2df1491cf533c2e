/*
 * wush.h - C ABI of the B200 (sm_100a) W4A4 WUSH linear-layer library.
 *
 * Method: "WUSH: Near-Optimal Adaptive Transforms for LLM Quantization"
 * (arXiv 2512.00956).  The online layer (Eq. 7, Sec. 5 "GPU Kernel Support") is
 *
 *     Y = sum_i  W~_(i)^T  q( T_wush(i)  X~_(i) )
 *
 * with block-diagonal transforms of block size d = g, q the round-to-nearest AbsMax
 * block quantiser over groups of g consecutive input channels (Sec. 3, "Block-
 * independent constraint"), and W~_(i) = q(T_xvsh(i) W_(i)) prepared offline
 * (Algorithm 2, RTN case) with T_xvsh = T_wush^-T (Eq. 6).
 *
 * Layout bridge.  The paper writes column vectors (X in R^{d_in x d_batch}, output
 * W^T X).  This library is row-major:  X[M,K], W[N,K], Y[M,N] = X W^T, with
 * M = d_batch, K = d_in, N = d_out, g = d, C = K/g.  T_(i) x on a column block is
 *     v[m, c*g + j] = sum_k T[c][j][k] * x[m, c*g + k].
 *
 * Formats.  MXFP4: g = 32, E2M1 codes, one E8M0 scale byte per block
 * (2^(byte-127), byte = 127 + floor(log2 AbsMax) - 2, clamped to [0,254]).
 * NVFP4: g = 16, E2M1 codes, one E4M3 scale byte per block and one fp32 scale per
 * tensor; with a = AbsMax of the block the scale byte is E4M3(round-nearest-even,
 * saturate 448) of (a / 6) / tensor_scale, elements are multiplied by
 * 1 / (float(scale byte) * tensor_scale) and rounded to E2M1 (nearest, ties to the
 * even code, saturate at 6, sign kept).  Two codes per byte, element 2t in the low
 * nibble.  NaN/Inf inputs are not detected (they saturate).
 *
 * Conventions for every entry point
 *   - all data pointers are DEVICE pointers owned by the caller unless a parameter is
 *     documented as "host"; the library does not allocate, free or retain them;
 *   - work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream) and the call returns without synchronising;
 *   - the return value is a wush_status_t: 0 on success, negative on error.
 *     Argument errors are found on the host before anything is launched, and then
 *     no output is touched.
 *   - base pointers must be 16-byte aligned; K must be a multiple of 64.
 *   - calls act on the CURRENT device of the calling thread; one-time launch set-up is
 *     remembered per device, so a process may use several devices (device ordinals 0..63).
 *   - entry points may be called from several host threads at once (the remembered set-up is
 *     written idempotently, the error text is per thread); calls that share an output buffer,
 *     a workspace or the built-in scratch of wush_calib_moments_static must be ordered by the caller.
 */
#ifndef WUSH_H_
#define WUSH_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  WUSH_OK = 0,
  WUSH_ERR_NULL = -1,      /* a required pointer is NULL */
  WUSH_ERR_SHAPE = -2,     /* non-positive size, K % g != 0, K % 64 != 0, N % 8 != 0 ... */
  WUSH_ERR_FORMAT = -3,    /* unknown format / layout, or g does not match the format */
  WUSH_ERR_ALIGN = -4,     /* a base pointer is not 16-byte aligned */
  WUSH_ERR_WORKSPACE = -5, /* workspace missing or smaller than wush_*_workspace_bytes() */
  WUSH_ERR_CUDA = -6,      /* a CUDA call or launch failed; see wush_last_cuda_error() */
  WUSH_ERR_TIMEOUT = -7,   /* a bounded device-side wait expired (wush_decode_status of a kernel's status word) */
  WUSH_ERR_DEVICE = -8     /* the current device is not compute capability 10.x */
} wush_status_t;

/* WUSH_MXFP4_CEIL is MXFP4 with the other common shared-exponent rule (the paper names only
 * "AbsMax" scaling, Sec. 3): byte = 127 + ceil(log2(AbsMax / 6)), the smallest exponent for
 * which no element of the block saturates, instead of 127 + floor(log2 AbsMax) - 2.  Codes
 * and scale bytes have the same meaning, so buffers quantised under either rule feed the
 * same GEMM; every call that takes a format accepts it with g = 32. */
typedef enum { WUSH_MXFP4 = 0, WUSH_NVFP4 = 1, WUSH_MXFP4_CEIL = 2 } wush_format_t;

/* Scale-byte layouts.
 *  LINEAR: scales[row][K/g], row-major.
 *  TILED : the layout the block-scaled tensor-core GEMM consumes.  Rows are padded to a
 *          multiple of 128 and scale columns to a multiple of 4; the byte of (row r,
 *          scale column kb) lives at
 *              ((r/128) * ceil(K/g/4) + kb/4) * 512 + (r%32)*16 + ((r%128)/32)*4 + kb%4.
 *          Padding bytes are never read for valid outputs and are left untouched.
 *          Size: wush_scale_bytes(rows, K, g, WUSH_SF_TILED). */
typedef enum { WUSH_SF_LINEAR = 0, WUSH_SF_TILED = 1 } wush_sf_layout_t;

typedef enum { WUSH_OUT_F32 = 0, WUSH_OUT_BF16 = 1 } wush_out_t;

const char* wush_status_string(int status);
/* Every wait inside the kernels is bounded (one to two seconds).  When one runs out, the kernel records a
 * diagnostic word in the int32 `status` buffer of the call (wush_gemm_fp4: its argument; wush_linear: the last
 * 16 bytes of the workspace), lets its outstanding copies land, frees what it holds and returns; the outputs
 * of that call are then undefined and the context stays usable.  The word is 0 when nothing expired, else
 * (role << 16) | index: role 0x06 / 0x07 / 0x08 = producer / MMA issuer / epilogue of the quantiser (0x04 / 0x05 =
 * producer / consumer of its warp-level variant; index = work item of the CTA),
 * 0x11..0x15 = producer, scale-copy wait, accumulator hand-over, epilogue, operand wait of the GEMM for
 * M > 128 (0x16 = that kernel found its shared-memory window misplaced and did no work),
 * 0x01..0x03 = producer, MMA issuer, epilogue of the GEMM for M <= 128.  The
 * caller copies the word to the host after synchronising; this helper maps it to WUSH_OK or WUSH_ERR_TIMEOUT. */
int wush_decode_status(int32_t word);
/* Text of the last CUDA error this library saw on the calling thread ("" if none). */
const char* wush_last_cuda_error(void);

/* Bytes of a scale buffer for `rows` rows in the given layout (0 on bad arguments). */
size_t wush_scale_bytes(int64_t rows, int64_t K, int g, wush_sf_layout_t sf);

/* ---------------------------------------------------------------------------------------
 * Online step 1 (Eq. 7 inner term, Sec. 5 "Fused WUSH + Quant kernel"):
 *   codes, scales = q( X_blk * T_c^T )  for every token row and every block c.
 *   X      bf16 [M,K] row-major.
 *   T      bf16 [K/g][g][g]; T[c][j][k] multiplies input channel c*g+k into output
 *          coordinate c*g+j (the activation-side transform T_wush of Eq. 5, stored as
 *          16-bit values, Sec. 3 "Costs for online inference").
 *   x_tensor_scale  fp32[1] on the device; NVFP4 only (static, chosen at calibration
 *          time), must be > 0; pass NULL for MXFP4.
 *   codes  uint8 [M, K/2];  scales uint8, layout `sf`.
 * Errors: NULL / SHAPE / FORMAT / ALIGN / CUDA.  M = 0 is a no-op returning WUSH_OK.
 * Stand-alone, this call has no status word (wush_linear has): its waits are bounded like all others, but an
 * expired one goes unreported and leaves part of the outputs unwritten.
 * For NVFP4 the tensor scale is read on the device when the kernel runs, so it may be the output of work
 * enqueued earlier on the same stream (wush_act_tensor_scale directly before this call, for example). */
int wush_quantize_act(const void* X, int64_t M, int64_t K, const void* T,
                      wush_format_t fmt, int g, const float* x_tensor_scale,
                      uint8_t* codes, uint8_t* scales, wush_sf_layout_t sf, void* stream);

/* The same step for NVFP4 with the tensor scale taken from THIS batch instead of from calibration
 * (the paper does not say how the NVFP4 tensor scale of online activations is obtained; the
 * static one above is this library's default, this is the alternative): a first pass finds
 * AbsMax over all M x K transformed values, the quantising pass uses AbsMax / (6 * 448)
 * (1 if the batch is all zero).  X is read twice.
 *   x_tensor_scale  fp32[2] on the device, WRITTEN: [0] = the scale used (pass it to
 *          wush_gemm_fp4), [1] = the AbsMax found (also the scratch word of the first pass).
 * g must be 16.  Errors as wush_quantize_act. */
int wush_quantize_act_dynamic(const void* X, int64_t M, int64_t K, const void* T, int g,
                              float* x_tensor_scale, uint8_t* codes, uint8_t* scales,
                              wush_sf_layout_t sf, void* stream);

/* The static NVFP4 activation tensor scale from calibration tokens (offline): the AbsMax pass of the call
 * above on Xc bf16 [B,K], without quantising.  out fp32[2] on the device, 8-byte aligned, WRITTEN:
 * [0] = AbsMax / (6 * 448) (1 if everything is zero), [1] = the AbsMax over all B x K transformed values.
 * g must be 16, B >= 1.  Errors: NULL / SHAPE / FORMAT / ALIGN / CUDA. */
int wush_act_tensor_scale(const void* Xc, int64_t B, int64_t K, const void* T, int g, float* out,
                          void* stream);

/* Offline weight preparation (Algorithm 2, RTN case, last line):
 *   W~ = q( W_blk * Tinv_c^T ),  Tinv = T_xvsh = T_wush^-T (Eq. 6) given in fp32.
 *   W      bf16 [N,K];  Tinv fp32 [K/g][g][g] (same index convention as T above).
 *   w_tensor_scale  fp32[1] on the device, WRITTEN for NVFP4: AbsMax of the whole
 *          transformed tensor / (6*448); ignored (may be NULL) for MXFP4.
 *   workspace       device scratch of at least wush_quantize_weight_workspace_bytes();
 *          contents on entry are irrelevant; must not be shared by overlapping calls.
 * The product is evaluated on tensor cores from an exact 3-way bf16 split of Tinv with
 * fp32 accumulation.  Errors as above plus WORKSPACE. */
int wush_quantize_weight(const void* W, int64_t N, int64_t K, const float* Tinv,
                         wush_format_t fmt, int g, float* w_tensor_scale,
                         uint8_t* codes, uint8_t* scales, wush_sf_layout_t sf,
                         void* workspace, size_t workspace_bytes, void* stream);
size_t wush_quantize_weight_workspace_bytes(int64_t N, int64_t K, wush_format_t fmt, int g);

/* Online step 2 (Eq. 7 outer sum): block-scaled FP4 GEMM on tcgen05 tensor cores,
 *   Y[m,n] = alpha * sum_c sx[m,c] * sw[n,c] * sum_{k in c} xq[m,k] * wq[n,k],
 *   alpha = 1 (MXFP4) or x_tensor_scale * w_tensor_scale (NVFP4), fp32 accumulation.
 *   Xq [M,K/2], Wq [N,K/2] packed codes; Xs, Ws scale bytes in TILED layout.
 *   Y  [M,N] row-major, fp32 or bf16 (`ydt`).  N must be a multiple of 8.
 *   status  optional int32[1] on the device: set to a non-zero diagnostic word if a
 *           bounded wait inside the kernel expired (then Y is undefined); may be NULL.
 * Errors: NULL / SHAPE / FORMAT / ALIGN / DEVICE / CUDA. */
int wush_gemm_fp4(const uint8_t* Xq, const uint8_t* Xs, const uint8_t* Wq, const uint8_t* Ws,
                  int64_t M, int64_t N, int64_t K, wush_format_t fmt, int g,
                  const float* x_tensor_scale, const float* w_tensor_scale,
                  void* Y, wush_out_t ydt, int32_t* status, void* stream);

/* The whole online layer (Eq. 7): wush_quantize_act into `workspace`, then wush_gemm_fp4,
 * both on `stream`.  Wcodes/Wscales come from wush_quantize_weight with WUSH_SF_TILED.
 * workspace: at least wush_linear_workspace_bytes(M, K, g) bytes, 16-byte aligned.  The
 * last 16 bytes of that region receive the GEMM's status word (see wush_gemm_fp4), the 16
 * bytes before them the activation tensor scale and AbsMax when x_tensor_scale is NULL.
 * NVFP4 with x_tensor_scale == NULL selects the per-batch tensor scale of
 * wush_quantize_act_dynamic (one more kernel, X read twice). */
int wush_linear(const void* X, int64_t M, int64_t K, const void* T,
                const uint8_t* Wcodes, const uint8_t* Wscales, int64_t N,
                const float* x_tensor_scale, const float* w_tensor_scale,
                wush_format_t fmt, int g, void* Y, wush_out_t ydt,
                void* workspace, size_t workspace_bytes, void* stream);
size_t wush_linear_workspace_bytes(int64_t M, int64_t K, int g);

/* One size for a workspace that serves every call of a layer with d_batch <= M tokens, d_out = N and d_in = K
 * (the arguments of the problem statement, Sec. 3 "Problem setup"): the largest of
 * wush_linear_workspace_bytes(M, K, g), wush_quantize_weight_workspace_bytes(N, K, fmt, g) and
 * wush_calib_moments_workspace_bytes(max(M, N), K, g) - calibration chunks of up to max(M, N) rows, which
 * covers the weight matrix itself.  0 on bad arguments. */
size_t wush_workspace_bytes(int64_t M, int64_t N, int64_t K, wush_format_t fmt, int g);

/* Offline calibration statistics (Algorithm 2, first line of the RTN loop):
 *   moments[c] += sum_t  x_{t,c}^T x_{t,c}   (unnormalised g x g second moment of block c)
 *   *count     += B
 *   Xc       bf16 [B,K] (calibration activations, or the weight matrix W[N,K] itself
 *            for the weight-side moment);  moments fp32 [K/g][g][g], accumulated in
 *            place so calibration can be fed in chunks; count int64[1] on the device.
 *   workspace device scratch of at least wush_calib_moments_workspace_bytes(B,K,g): the per-CTA partial sums
 *            of the first kernel, added up in a fixed order by the second (no floating-point atomics).
 * The reduction order is fixed, so results are run-to-run identical.  count must be 8-byte aligned.
 * Sums are fp32: within 1e-5 of the exact sums (relative to the largest entry of a block) up to at least 2.6e5 rows.
 * This call has no status word: should one of its bounded waits expire, the affected moments are written
 * as NaN, so a failed call cannot be mistaken for a result. */
int wush_calib_moments(const void* Xc, int64_t B, int64_t K, int g, float* moments,
                       int64_t* count, void* workspace, size_t workspace_bytes, void* stream);
size_t wush_calib_moments_workspace_bytes(int64_t B, int64_t K, int g);

/* Offline transform construction (Algorithm 1 for every block, and the pairing of Eq. 6):
 *   from the UNNORMALISED second-moment sums of the weights (mom_w, over rows_w = d_out rows) and of
 *   the calibration activations (mom_x, over rows_x = d_batch tokens), both fp32 [K/g][g][g] as
 *   wush_calib_moments produces them, compute per block
 *       W', X' = lower Cholesky factors of the damped moments  M + lambda * tr(M)/g * I,
 *       U S V^T = SVD(W'^T X'),   T_wush = H S^-1/2 U^T W'^T   (H: normalised Sylvester-Hadamard),
 *   T     <- bf16(T_wush)          [K/g][g][g]   (input of wush_quantize_act / wush_linear)
 *   Tinv  <- (T)^-T in fp32        [K/g][g][g]   (= T_xvsh for the stored T; input of wush_quantize_weight)
 *   info  optional int32[K/g] on the device: 0 = ok, 1 = a Cholesky pivot was not positive,
 *         2 = the Jacobi SVD did not converge, 3 = T was singular.  May be NULL.
 * The SVD is unique only up to signs and the order of equal singular values (Lemma A.1); the
 * convention here is: singular values descending, each row of U^T W'^T signed so that its
 * largest-magnitude entry is positive.  fp64 arithmetic throughout.
 * Errors: NULL / SHAPE (incl. lambda < 0, rows <= 0) / FORMAT / ALIGN / CUDA. */
int wush_build_transforms(const float* mom_w, int64_t rows_w, const float* mom_x, int64_t rows_x,
                          int64_t K, int g, float lambda, void* T, float* Tinv, int32_t* info,
                          void* stream);
/* The same with a choice of transform: WUSH_KIND_WUSH (the call above), WUSH_KIND_WUS, the ablation of
 * Sec. 6 / Table 1 "WUSH without Hadamard", T = S^-1/2 U^T W'^T, or one of the two fixed transforms described
 * at the enum.  Errors as above; FORMAT for another kind. */
typedef enum {
  WUSH_KIND_WUSH = 0,
  WUSH_KIND_WUS = 1,
  /* The two data-independent comparison transforms of Sec. 5 ("H + Quant", "None + Quant") and Table 1: the same
   * normalised Sylvester-Hadamard matrix H[j][k] = (-1)^popcount(j & k) / sqrt(g) for every block, or the
   * identity.  mom_w, mom_x, rows_w, rows_x and lambda are ignored (the pointers may be NULL); T receives the
   * bf16-rounded matrix replicated K/g times, Tinv the inverse-transpose of those stored values. */
  WUSH_KIND_HADAMARD = 2,
  WUSH_KIND_IDENTITY = 3
} wush_transform_kind_t;
int wush_build_transforms_kind(const float* mom_w, int64_t rows_w, const float* mom_x, int64_t rows_x,
                               int64_t K, int g, float lambda, wush_transform_kind_t kind, void* T,
                               float* Tinv, int32_t* info, void* stream);
/* Weight-side partners of given activation-side transforms (Eq. 6): Tinv[c] = (T[c])^-T for every block,
 * fp64 Gauss-Jordan with partial pivoting, result in fp32.  T bf16 [K/g][g][g] (any transforms: a shared
 * Hadamard matrix, the identity, user-supplied ones), Tinv fp32 [K/g][g][g], info optional int32[K/g]
 * (0 = ok, 3 = singular).  Errors: NULL / SHAPE / FORMAT / ALIGN / CUDA. */
int wush_invert_transforms(const void* T, int64_t K, int g, float* Tinv, int32_t* info, void* stream);

/* Offline weight preparation, GPTQ case of Algorithm 2: the transforms are built block by block from the UPDATED
 * weights, and every block's quantisation error is spread first inside the block (the GPTQ subroutine on the
 * transformed block with the transformed Hessian) and then over all later blocks (W_(j) += L_(j,i) L_(i,i)^-1 E_(i)),
 * with L L^T the Cholesky factorisation of the inverse of the damped Hessian H + lambda * tr(H)/K * I,
 * H = Xc^T Xc / B.  Replaces wush_calib_moments + wush_build_transforms + wush_quantize_weight for a layer; the
 * online calls are the same.
 *   W      bf16 [N,K];  Xc bf16 [B,K] calibration activations (the layer's inputs).
 *   lambda damping ratio, > 0 (used for the Hessian and inside Algorithm 1).
 *   w_tensor_scale  fp32[1] on the device, INPUT, NVFP4 only: the tensor scale has to be fixed before the first
 *          block is quantised while the weights still change, so the caller chooses it (for example the value
 *          wush_quantize_weight returns for the same layer); NULL for MXFP4.
 *   T      bf16 [K/g][g][g] WRITTEN (activation-side transforms, as wush_build_transforms);
 *   Tinv   fp32 [K/g][g][g] WRITTEN;  codes [N,K/2], scales in layout `sf` WRITTEN.
 *   info   optional int32[K/g]: 0 ok, 1..3 as wush_build_transforms, 4 = the block's transformed Hessian could not
 *          be factorised, 5 = the damped Hessian could not be factorised.
 *   workspace  at least wush_gptq_workspace_bytes(N, K, g) bytes, 256-byte aligned: fp64 copies of W (N x K) and
 *          of two K x K matrices and eight N x g blocks - about 8 (N K + 2 K^2 + 8 N g) bytes.
 * The scale of a block is fixed when its turn comes, from its current values; each coordinate is rounded to fp32
 * before it is converted, as in the RTN quantiser.  fp64 arithmetic throughout, fixed summation orders (results
 * are run-to-run identical).  A sequential offline solver: about 2 K + 7 K/g kernel launches (28672 x 8192 with 4096
 * calibration tokens: about 10 s on a B200).
 * Errors: NULL / SHAPE (incl. lambda <= 0, B <= 0, K > 32768) / FORMAT / ALIGN / WORKSPACE / CUDA. */
int wush_gptq_quantize_weight(const void* W, int64_t N, int64_t K, const void* Xc, int64_t B,
                              wush_format_t fmt, int g, float lambda, const float* w_tensor_scale,
                              void* T, float* Tinv, uint8_t* codes, uint8_t* scales, wush_sf_layout_t sf,
                              int32_t* info, void* workspace, size_t workspace_bytes, void* stream);
size_t wush_gptq_workspace_bytes(int64_t N, int64_t K, int g);

/* wush_calib_moments without a workspace argument.  (No counterpart in the paper: this is
 * a packaging variant of the call above, added for hosts where this library must not and
 * cannot obtain device memory at call time - for example a serving process whose allocator
 * has claimed the whole HBM for its own arena and has no API to lend a slice to a plug-in,
 * or a runtime that forbids allocation after start-up.  Such a caller has nowhere to get
 * the scratch buffer the normal entry point asks for.)
 *
 * The per-split partial sums live in a fixed array of WUSH_STATIC_SCRATCH_BYTES inside the
 * library image; every GPU that loads the library carries that array until the process
 * exits.  Inputs and outputs are still the caller's.  The call allocates nothing and frees
 * nothing.  Limits and rules:
 *   - K * g * 4 bytes (one set of partial sums) must fit in the array, otherwise
 *     WUSH_ERR_WORKSPACE is returned and nothing is launched; larger B only lowers the number
 *     of token splits that run in parallel (down to one), never the result;
 *   - the first call on each device resolves the array's device address (a CUDA runtime
 *     symbol lookup, done once per device with that device current); make that first call
 *     during start-up, before any stream capture;
 *   - all calls on a device share the one array.  It keeps whatever the previous call left;
 *     nothing in it needs clearing because every call overwrites the part it reads.  Two
 *     calls whose kernels overlap on the GPU (different streams, no ordering) race on it:
 *     serialise them;
 *   - results match wush_calib_moments to fp32 summation-order differences (identical when
 *     both use the same number of splits), and are run-to-run identical. */
#define WUSH_STATIC_SCRATCH_BYTES (4u << 20)
int wush_calib_moments_static(const void* Xc, int64_t B, int64_t K, int g, float* moments,
                              int64_t* count, void* stream);

/* ----------------------------------------------------------------- diagnostic exports */
/* The block quantiser q(.) alone on fp32 input V[R,K] (same outputs as above). */
int wush_quantize_f32(const float* V, int64_t R, int64_t K, wush_format_t fmt, int g,
                      const float* tensor_scale, uint8_t* codes, uint8_t* scales,
                      wush_sf_layout_t sf, void* stream);
/* The NVFP4 scale byte is E4M3((AbsMax / 6) / tensor_scale) with both divisions correctly rounded.  The kernels
 * take two shortcuts that must give the same byte: (a) inside AbsMax in [2^-50, 2^50] and tensor_scale in
 * [2^-40, 2^40] the divisions are evaluated without the IEEE division sequence (reciprocal of the divisor, two
 * fused multiply-add corrections); (b) where AbsMax * RN(1 / (6 tensor_scale)) is clear of every E4M3 rounding
 * boundary by more than its own error, that product is converted directly.  This call checks both on the device:
 * for each of the n values b (fp32, device array, normal, in [2^-40, 2^40]) it compares, for EVERY fp32 x in
 * [2^-60, 2^60], x / b by (a) with the IEEE quotient, and the scale byte of a block with AbsMax = x under tensor
 * scale b as the kernels compute it with the byte of the IEEE sequence; mismatches[i] (uint64, device array)
 * receives the number of x for which either differs (expected: all zero).  A few ms per value. */
int wush_check_division(const float* divisors, int n, uint64_t* mismatches, void* stream);
/* Test hook for the persistent GEMM (M > 128): use at most `clusters` two-CTA clusters in later calls on the
 * current device (0 = as many as fit, the default; the setting is per device, shared by all threads).  With few clusters even a small problem
 * gives every cluster several tiles in a row, which is how the tests reach the hand-over between tiles
 * (accumulator drained while the next tile's loads run) without a full-size input.  Results never depend
 * on it.  Returns the previous value. */
int wush_debug_gemm_clusters(int clusters);
/* Test hook for the activation quantiser.  By default (0) wush_quantize_act / wush_quantize_act_dynamic /
 * wush_linear run the kernel that does the block products on the tcgen05 tensor cores; 64 or 128 selects the
 * warp-level streaming kernel (the one the weight side uses, and the fall-back) with that many token rows per
 * tile, for later calls on the current device (a per-device setting).  The tests use it to run ragged token counts
 * and channel tails through every instantiation without full-size inputs.  Results never depend on it.
 * Returns the previous value, or WUSH_ERR_SHAPE for another value. */
int wush_debug_quantiser_rows(int rows);
/* Test hook for the error path: the next wush_linear call on the current device (whichever thread makes it) leaves the
 * tile of work item `item` of its quantiser kernel unrequested (one call only; -1 cancels).  The consumers'
 * bounded wait for that tile (about a second) then expires, the status word is set, both kernels of the
 * call still complete and the next call works as usual.  Nothing faults and nothing waits without a bound. */
int wush_debug_drop_tile(int item);
/* The block transform alone: V[M,K] fp32 = X_blk * T_c^T, same arithmetic as
 * wush_quantize_act uses before quantising. */
int wush_transform_act_f32(const void* X, int64_t M, int64_t K, const void* T, int g,
                           float* V, void* stream);
/* Same for the weight side (fp32 Tinv, 3-way split). */
int wush_transform_weight_f32(const void* W, int64_t N, int64_t K, const float* Tinv, int g,
                              float* V, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* WUSH_H_ */
