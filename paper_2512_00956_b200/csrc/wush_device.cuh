// Device-side helpers shared by the kernels of libwush: scale-layout indexing, the
// E2M1 / E8M0 / E4M3 block quantiser q(.) of Sec. 3 ("Block-independent constraint"),
// and the warp-level bf16 tensor-core instruction used for the g x g block products.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp4.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace wush {

constexpr int kFmtMX = 0;   // MXFP4: g = 32, E8M0 scale
constexpr int kFmtNV = 1;   // NVFP4: g = 16, E4M3 scale + fp32 tensor scale

// Byte offset of the scale of (row r, scale column kb) in a buffer with KB scale columns.
// layout 0: [rows][KB];  layout 1: 128-row x 4-column tiles of 512 bytes, the order the
// block-scaled MMA reads from tensor memory (32 lanes x 16 bytes, four 32-row groups
// interleaved at 4-byte granularity).
__host__ __device__ __forceinline__ int64_t sf_offset(int layout, int64_t r, int64_t kb, int64_t KB) {
  if (layout == 0) return r * KB + kb;
  const int64_t ktiles = (KB + 3) >> 2;
  return ((r >> 7) * ktiles + (kb >> 2)) * 512 + (r & 31) * 16 + ((r & 127) >> 5) * 4 + (kb & 3);
}

// ---- E2M1: round to nearest (ties to the even code), saturate at 6, keep the sign.
// Packs 8 fp32 values into 8 nibbles, element 0 in the lowest nibble.
__device__ __forceinline__ uint32_t pack_e2m1x8(const float (&u)[8]) {
  uint32_t w = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_fp4x2_storage_t b =
        __nv_cvt_float2_to_fp4x2(make_float2(u[2 * i], u[2 * i + 1]), __NV_E2M1, cudaRoundNearest);
    w |= static_cast<uint32_t>(b) << (8 * i);
  }
  return w;
}

// Same packing, written so that the four conversions and the byte merge are five instructions:
// cvt.rn.satfinite.e2m1x2.f32 d, a, b puts a in the high nibble and b in the low one.
__device__ __forceinline__ uint32_t pack_e2m1x8_fast(const float (&u)[8]) {
  uint32_t w;
  asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
      "mov.b32 %0, {b0, b1, b2, b3};\n\t}"
      : "=r"(w)
      : "f"(u[0]), "f"(u[1]), "f"(u[2]), "f"(u[3]), "f"(u[4]), "f"(u[5]), "f"(u[6]), "f"(u[7]));
  return w;
}

// the register pair {m, m}: second operand of the packed multiply below
__device__ __forceinline__ uint64_t pair_of(float m) {
  uint64_t p;
  asm("mov.b64 %0, {%1, %1};" : "=l"(p) : "f"(m));
  return p;
}
// (a, b) * (m, m) with one packed fp32 instruction (round to nearest, no flush), multiplier given as pair_of(m)
__device__ __forceinline__ void mul2_rn(float& a, float& b, uint64_t mm) {
  asm("{\n\t.reg .b64 v;\n\t"
      "mov.b64 v, {%0, %1};\n\t"
      "mul.rn.f32x2 v, v, %2;\n\t"
      "mov.b64 {%0, %1}, v;\n\t}"
      : "+f"(a), "+f"(b)
      : "l"(mm));
}
// (x, y) = (a, b) * (m, m), results in registers of their own
__device__ __forceinline__ void mul2_rn_to(float& x, float& y, float a, float b, uint64_t mm) {
  asm("{\n\t.reg .b64 v;\n\t"
      "mov.b64 v, {%2, %3};\n\t"
      "mul.rn.f32x2 v, v, %4;\n\t"
      "mov.b64 {%0, %1}, v;\n\t}"
      : "=f"(x), "=f"(y)
      : "f"(a), "f"(b), "l"(mm));
}
// (a, b) * (m, m) with one packed fp32 instruction (round to nearest, no flush)
__device__ __forceinline__ void mul2_rn(float& a, float& b, float m) {
  asm("{\n\t.reg .b64 v, s;\n\t"
      "mov.b64 v, {%0, %1};\n\t"
      "mov.b64 s, {%2, %2};\n\t"
      "mul.rn.f32x2 v, v, s;\n\t"
      "mov.b64 {%0, %1}, v;\n\t}"
      : "+f"(a), "+f"(b)
      : "f"(m));
}

// ---- MXFP4 scale: e = clamp(floor(log2 amax) - 2, -127, 127); returns the E8M0 byte and
// the exact fp32 multiplier 2^-e.  amax is finite and non-negative.
// ceil_rule != 0 selects e = ceil(log2(amax / 6)) instead, the smallest exponent that saturates
// nothing: with amax = 1.f * 2^E that is E - 2 when the fraction 1.f <= 1.5 and E - 1 otherwise,
// i.e. the floor-rule exponent plus (mantissa field > 0x400000).
__device__ __forceinline__ void mx_scale(float amax, uint32_t& byte, float& mult, int ceil_rule = 0) {
  const uint32_t bits = __float_as_uint(amax);
  int e = static_cast<int>((bits >> 23) & 0xFF) - 127 - 2;                    // zero/subnormal -> -129
  if (ceil_rule) e += ((bits & 0x7FFFFFu) > 0x400000u) ? 1 : 0;
  e = e < -127 ? -127 : e;                                                   // e <= 126 for finite input
  byte = static_cast<uint32_t>(e + 127);
  mult = __uint_as_float(static_cast<uint32_t>(127 - e) << 23);               // 2^-e, biased 2..254
}

__device__ __forceinline__ float e4m3_to_float(uint32_t byte) {
  __half_raw h = __nv_cvt_fp8_to_halfraw(static_cast<__nv_fp8_storage_t>(byte), __NV_E4M3);
  return __half2float(__half(h));
}

// NVFP4 tensor scale from the AbsMax of the whole tensor: AbsMax / (6 * 448), one fp32 division;
// 1 for an all-zero tensor (any positive value then yields the same all-zero codes).
__device__ __forceinline__ float nv_tensor_scale(float amax) {
  return amax == 0.0f ? 1.0f : __fdiv_rn(amax, 2688.0f);
}

// ---- NVFP4 scale.  Single-rounded fp32 steps, in this order and with no contraction:
//   r = (amax / 6) / ts ;  byte = E4M3(r) ;  d = float(byte) * ts ;  mult = d == 0 ? 0 : 1 / d.
// The two halves separately: the scale byte of a block, and the multiplier that belongs to a scale byte.
// The multiplier depends on (byte, ts) only, so a kernel may tabulate it for the 128 byte values once.
__device__ __forceinline__ uint32_t nv_scale_byte(float amax, float ts) {
  const float r = __fdiv_rn(__fdiv_rn(amax, 6.0f), ts);
  return static_cast<uint32_t>(__nv_cvt_float_to_fp8(r, __NV_SATFINITE, __NV_E4M3));
}

// x / b, correctly rounded, without the branchy IEEE division sequence: y = RN(1 / b) is given, one FMA
// step makes the quotient faithful, a second one rounds it correctly (Markstein's division).  Valid while no
// intermediate leaves the normal range; the callers below guard that.  wush_check_division compares it with
// __fdiv_rn over all x of the guarded range for any divisors it is given.
__device__ __forceinline__ float div_rn_fma(float x, float b, float y) {
  float q = __fmul_rn(x, y);
  float r = __fmaf_rn(-b, q, x);
  q = __fmaf_rn(r, y, q);
  r = __fmaf_rn(-b, q, x);
  return __fmaf_rn(r, y, q);
}
constexpr float kRcp6 = 0.16666667163372040f;        // RN(1/6) = 0x3E2AAAAB
// Per-kernel constants of the fast scale paths: rts = RN(1 / ts) and c = RN(RN(1/6) * rts) ~ 1 / (6 ts), usable
// while ts lies in [2^-40, 2^40]
struct NvScaleFast {
  float ts, rts, c;
  bool ts_ok;
};
__device__ __forceinline__ NvScaleFast nv_scale_fast(float t) {
  NvScaleFast f;
  f.ts = t;
  f.rts = __frcp_rn(t);
  f.c = __fmul_rn(kRcp6, f.rts);
  f.ts_ok = (t >= 0x1p-40f && t <= 0x1p40f);
  return f;
}
// The pinned sequence with the divisions done by FMAs where that is exact (blocks with amax in [2^-50, 2^50], both
// intermediates then stay far inside the normal range), the IEEE ones otherwise - zero blocks included.
__device__ __forceinline__ uint32_t nv_scale_byte_slow(float amax, const NvScaleFast& f) {
  float r;
  if (f.ts_ok && amax >= 0x1p-50f && amax <= 0x1p50f) r = div_rn_fma(div_rn_fma(amax, 6.0f, kRcp6), f.ts, f.rts);
  else r = __fdiv_rn(__fdiv_rn(amax, 6.0f), f.ts);
  return static_cast<uint32_t>(__nv_cvt_float_to_fp8(r, __NV_SATFINITE, __NV_E4M3));
}
// The same byte as nv_scale_byte(amax, f.ts).  The byte only depends on which E4M3 rounding interval r falls into, so
// an approximation of r decides it whenever it is clear of every interval boundary: r' = RN(amax * c) lies within
// 4 ulp of the pinned r (c carries 1.5 ulp, the product half an ulp, the pinned r one ulp against the exact
// quotient).  In the normal range of E4M3 (r >= 2^-6) the boundaries are the values whose low 20 mantissa bits
// are 0x80000; r' further than 16 ulp from that pattern gives the pinned byte by conversion (above 448 everything
// saturates, and the boundaries 432 and 464 on the way there have the same pattern).  Anything else - about one
// block in 30000, the subnormal range, zero blocks - takes the pinned sequence.  wush_check_division compares the
// two for every fp32 amax.
__device__ __forceinline__ uint32_t nv_scale_byte(float amax, const NvScaleFast& f) {
  const float rf = __fmul_rn(amax, f.c);
  const uint32_t low = __float_as_uint(rf) & 0xFFFFFu;
  if (f.ts_ok && rf >= 0x1.01p-6f && (low - 0x7FFF0u) >= 0x20u)
    return static_cast<uint32_t>(__nv_cvt_float_to_fp8(rf, __NV_SATFINITE, __NV_E4M3));
  return nv_scale_byte_slow(amax, f);
}
__device__ __forceinline__ float nv_mult_of_byte(uint32_t byte, float ts) {
  const float d = __fmul_rn(e4m3_to_float(byte), ts);
  return (d == 0.0f) ? 0.0f : __frcp_rn(d);
}
__device__ __forceinline__ void nv_scale(float amax, float ts, uint32_t& byte, float& mult) {
  byte = nv_scale_byte(amax, ts);
  mult = nv_mult_of_byte(byte, ts);
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// D = A * B (no accumulator input: the zero operand costs no register moves)
__device__ __forceinline__ void mma_bf16_16816_first(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                     uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%10,%10,%10,%10};\n"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.0f));
}

// transpose an 8x8 matrix of 16-bit elements held one 32-bit register per lane
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}

// fetch a TMA descriptor (a __grid_constant__ kernel parameter) into the descriptor cache ahead of its first use
__device__ __forceinline__ void prefetch_tensormap(const void* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ uint4 ld_global_nc_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

}  // namespace wush
