// Streaming variant of the fused block transform + quantise kernel (Eq. 7 inner term) used by
// the online path: the same arithmetic as transform_quant.cu, restructured so that HBM stays
// busy.
//
//  * Persistent CTAs (one per SM): 1 producer warp + 16 consumer warps.  The producer streams
//    ROWS-row x 128-channel tiles of X into a shared-memory ring of 128 KB with TMA (two
//    128-byte-wide boxes per tile, 128-byte swizzle, no multicast): 4 stages of 128 rows, or, for
//    small problems, 8 stages of 64 rows - finer work items, so the first one lands sooner and the
//    CTAs finish closer together.
//  * A work item is (128-channel panel, ROWS-row block); a CTA takes a contiguous run of items in
//    panel-major order, so the panel rarely changes.  Each consumer warp owns one 16-row slice
//    and two (ROWS = 128) or one (ROWS = 64) of the panel's four 32-channel super-blocks, and keeps
//    the MMA B-fragments of those transforms in REGISTERS for as long as the panel stays the same.
//  * A operands: g = 32 uses ldmatrix.x4 (its destination registers are the MMA operand quad);
//    g = 16 reads 16 contiguous bytes per lane and row with a permuted contraction index.
//  * Output permutation: MMA column slot (tile t, n) carries transform row 8*c(n/2) + 2*t + n%2
//    with c = (0,2,1,3), so every lane owns 8 consecutive outputs = 4 code bytes; with two
//    super-blocks per warp one shuffle with lane^2 makes that 8 contiguous bytes and a row's 32
//    bytes leave as one full sector per quad.
//  * Interior items (all rows and super-blocks present) run a copy of the item body without predicates.
#include <cuda.h>

#include <type_traits>

#include "wush_device.cuh"
#include "wush_host.h"

namespace wush {

// Tile geometry.  ROWS = 128: 16 warps = 8 row slices x 2 pairs of super-blocks, 4 ring stages of 32 KB.
// ROWS = 64 (small problems: finer work items, the first one lands sooner, CTAs end closer together):
// 16 warps = 4 row slices x 4 super-blocks, 8 stages of 16 KB.  Bytes in flight are the same.
constexpr int SQ_RING_BYTES = 128 * 1024;
constexpr int SQ_MAX_STAGES = 8;
constexpr int SQ_SMALL = 5;          // fewer 128-row items per CTA than this: use 64-row tiles (measured: 3.5 per
                                     // CTA gains 7-25 %, 7 per CTA loses 6 %, large problems are unchanged)
constexpr int SQ_CONSUMERS = 16;
constexpr int SQ_THREADS = (SQ_CONSUMERS + 1) * 32;
// ring | full[8] empty[8] barriers (128 B) | abort flag (64 B) | NVFP4 multiplier table (512 B); 1 KiB alignment slack
constexpr int SQ_SMEM = SQ_RING_BYTES + 1024 + 128 + 64 + 512;

__device__ __forceinline__ uint32_t sq_smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ bool sq_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t sq_timer() { uint64_t t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
// bounded wait (about one second); false on expiry or when another role has aborted
__device__ __forceinline__ bool sq_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < 2048; ++i)
    if (sq_try_wait(bar, parity)) return true;
  const uint64_t t0 = sq_timer();
  while (true) {
    for (int i = 0; i < 64; ++i)
      if (sq_try_wait(bar, parity)) return true;
    if (*abort_flag != 0 || sq_timer() - t0 > 1000000000ull) return false;
  }
}
__device__ __forceinline__ uint4 sq_lds128(uint32_t addr) {          // 128-bit load from a 32-bit shared address
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float sq_lds_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}
// four 8x8 matrices of 16-bit elements, one row address per lane: the result is the A operand of m16n8k16
__device__ __forceinline__ uint4 sq_ldmatrix_x4(uint32_t addr) {
  uint4 v;
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ bool sq_elect() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
  return pred != 0;
}

// AMAX = true: the same tile walk and the same products, but instead of quantising, the AbsMax of everything
// computed is folded into *ts_out (read as the uint32 bit pattern of a non-negative float, atomicMax): the
// first pass of the per-batch NVFP4 tensor scale.  codes / scales are not touched.
// NSPLIT = 3: the weight side (Algorithm 2, last line).  Tsrc is then the fp32 T_xvsh; every entry is split
// exactly into three bf16 terms (hi + mid + lo) when the fragments are loaded, and the three partial
// products are accumulated smallest first.  Needs ROWS = 64 (three sets of fragments per super-block).
template <int G, bool AMAX = false, int ROWS = 128, int NSPLIT = 1>
__global__ void __launch_bounds__(SQ_THREADS, 1)
tq_stream_kernel(const __grid_constant__ CUtensorMap mapX, const void* __restrict__ Tsrc, int64_t M, int64_t K,
                 const float* __restrict__ ts_ptr, uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                 int sf_layout, int num_rb, int num_items, int32_t* __restrict__ status, int clear_status,
                 const uint32_t* __restrict__ amax_in, float* __restrict__ ts_out, int mx_ceil, int drop_item) {
  constexpr int FMT = (G == 32) ? kFmtMX : kFmtNV;
  static_assert(NSPLIT == 1 || (NSPLIT == 3 && ROWS == 64), "three-way split needs one super-block per warp");
  constexpr int SQ_ROWS = ROWS;
  const __nv_bfloat16* T = reinterpret_cast<const __nv_bfloat16*>(Tsrc);      // NSPLIT = 1
  const float* Tf = reinterpret_cast<const float*>(Tsrc);                     // NSPLIT = 3
  constexpr int NQ = ROWS / 64;                      // super-blocks per consumer warp
  constexpr int SLICES = ROWS / 16;                  // 16-row slices per tile
  constexpr int SQ_BOX_BYTES = ROWS * 128;           // one TMA box: ROWS rows x 64 channels
  constexpr int SQ_STAGE_BYTES = 2 * SQ_BOX_BYTES;   // a 128-channel panel
  constexpr int SQ_STAGES = SQ_RING_BYTES / SQ_STAGE_BYTES;
  extern __shared__ uint8_t sq_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(sq_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + SQ_RING_BYTES);
  uint64_t* empty_bar = full_bar + SQ_MAX_STAGES;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(empty_bar + SQ_MAX_STAGES);

  // NVFP4: 1 / (float(scale byte) * ts) for all 128 scale bytes, the same two roundings as nv_scale, done once
  float* nv_mult = reinterpret_cast<float*>(smem + SQ_RING_BYTES + 128 + 64);
  const bool nv_quant = (FMT == kFmtNV) && !AMAX;
  const bool nv_dynamic = nv_quant && amax_in != nullptr;
  float ts = 1.0f;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 32) prefetch_tensormap(&mapX);
  if (threadIdx.x == 0) {
    for (int s = 0; s < SQ_STAGES; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(sq_smem_u32(&full_bar[s])), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(sq_smem_u32(&empty_bar[s])), "r"(SQ_CONSUMERS));
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // Launched as a programmatic dependent (wush_linear does), everything above ran while the previous kernel
  // of the stream was still draining; nothing it wrote or still reads may be touched before this point.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // the status word is only ever set after a bounded wait of about a second has expired, so clearing it
  // here cannot race with a report; it saves wush_linear a separate memset between kernels
  if (clear_status && blockIdx.x == 0 && threadIdx.x == 0 && status != nullptr) *status = 0;
  if (nv_quant) {
    // The tensor scale is read only here, after the dependency wait: the static one may have been written by
    // the kernel just before this one on the stream (wush_act_tensor_scale followed by the first layer call),
    // the per-batch one always is (the AbsMax pass).
    ts = nv_dynamic ? nv_tensor_scale(__uint_as_float(*amax_in)) : *ts_ptr;
    if (threadIdx.x < 128) nv_mult[threadIdx.x] = nv_mult_of_byte(threadIdx.x, ts);
    if (nv_dynamic && blockIdx.x == 0 && threadIdx.x == 0 && ts_out != nullptr) *ts_out = ts;
    __syncthreads();
  }
  // let a programmatic dependent (the GEMM of wush_linear) be scheduled as SMs free up; it still waits
  // for this whole grid before reading the codes
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // contiguous run of items for this CTA; item -> (panel, row block), panel-major
  const int item_begin = (int)(((int64_t)num_items * blockIdx.x) / gridDim.x);
  const int item_end = (int)(((int64_t)num_items * (blockIdx.x + 1)) / gridDim.x);
  const int total_sb = (int)(K >> 5);

  if (warp == SQ_CONSUMERS) {
    // ------------------------------------------------------------------ producer warp
    int n = 0;
    int panel = item_begin / num_rb, rb = item_begin % num_rb;
    for (int it = item_begin; it < item_end; ++it, ++n) {
      const int s = n % SQ_STAGES;
      const uint32_t ph = (n / SQ_STAGES) & 1;
      if (!__all_sync(0xffffffffu, sq_wait(sq_smem_u32(&empty_bar[s]), ph ^ 1, abort_flag))) {
        if (lane == 0) { if (*abort_flag == 0 && status) atomicExch(status, 0x40000 | n); *abort_flag = 1; }
        break;
      }
      const int nsb = min(4, total_sb - panel * 4);
      // drop_item (a test hook, -1 in production): this item's tile is never requested, so the consumers'
      // bounded wait for it runs out and the kernel leaves through its error path
      if (it != drop_item && sq_elect()) {
        const uint32_t bar = sq_smem_u32(&full_bar[s]);
        const int nbox = nsb >> 1;                       // 64-channel (128-byte) boxes; K % 64 == 0
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(nbox * SQ_BOX_BYTES) : "memory");
        for (int bx = 0; bx < nbox; ++bx) {
          const uint32_t dst = sq_smem_u32(smem + s * SQ_STAGE_BYTES + bx * SQ_BOX_BYTES);
          asm volatile(
              "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
              ::"r"(dst), "l"(&mapX), "r"((panel * 2 + bx) * 64), "r"(rb * SQ_ROWS), "r"(bar) : "memory");
        }
      }
      __syncwarp();
      if (++rb == num_rb) { rb = 0; ++panel; }
    }
    if (*abort_flag != 0) {
      // a wait expired somewhere: let every tile that was requested land before the CTA exits
      for (int k = max(0, n - SQ_STAGES); k < n; ++k) {
        const uint64_t t0 = sq_timer();
        while (!sq_try_wait(sq_smem_u32(&full_bar[k % SQ_STAGES]), (k / SQ_STAGES) & 1))
          if (sq_timer() - t0 > 500000000ull) break;
      }
    }
  } else {
    // ------------------------------------------------------------------ consumer warps
    const int gid = lane >> 2, tig = lane & 3;
    const int mt = warp % SLICES;             // 16-row slice of the tile
    const int wsb = (warp / SLICES) * NQ;     // first of this warp's NQ super-blocks (of the panel's four)
    // Two ways to fetch the A operands.  g = 32: ldmatrix, whose four destination registers ARE the operand
    // quad of mma.sync (standard fragment layouts; MMA row slot gid is tile row 16*mt + gid) - the 128-bit
    // loads of the other scheme cost about 29 register moves per 16 x 32 unit to interleave two rows into
    // quads.  g = 16: the scale arithmetic, not the instruction count, bounds that instantiation and the
    // longer ldmatrix latency measured slower, so it keeps the permuted contraction index: every lane reads 16
    // contiguous bytes of its two rows and of a transform row; row slot gid reads tile row 16*mt + pi(gid),
    // pi = (0,4,1,5,2,6,3,7), so that the two rows of a quarter-warp fall into disjoint bank halves.
    constexpr bool LDSM = (G == 32);
    const int prow = LDSM ? 16 * mt + gid : 16 * mt + ((gid & 1) << 2) + (gid >> 1);
    const int nchunk = (((gid >> 1) & 1) << 1) | (gid >> 2);  // c(gid/2): chunk of the column slot this lane feeds
    const int64_t KB = K / G;
    float seen = 0.0f;                         // AMAX: running maximum of this lane
    const uint32_t nv_mult_u32 = sq_smem_u32(nv_mult);
    const NvScaleFast nvf = nv_scale_fast(ts);                 // NVFP4: reciprocal of the tensor scale for the branch-free divisions

    uint4 tf[NSPLIT][NQ][4];                  // B fragments of this warp's transforms, kept across items
                                              // (NSPLIT = 3: [0] = lo, [1] = mid, [2] = hi terms)
    int cur_panel = -1;
    int n = 0;
    int panel = item_begin / num_rb, rb = item_begin % num_rb;
    const int KB32 = (int)KB;
    const int ktiles = (KB32 + 3) >> 2;
    const int64_t code_pitch = K >> 1;
    // Everything that does not change from item to item is worked out once: the shared-memory addresses of
    // this lane's two 16-byte pieces per super-block (32-bit, relative to the stage), and the steps by which
    // the output pointers advance when the row block does.
    // ldmatrix.x4: lane l addresses row (l & 7) + 8 * ((l >> 3) & 1) of the warp's 16-row slice and the 16-byte
    // chunk c0 + (l >> 4) of its 128-byte box row; chunk index XORed with (row & 7) by the TMA swizzle
    const int lm_row = LDSM ? 16 * mt + (lane & 7) + ((lane >> 3) & 1) * 8 : prow;
    const uint32_t x_base = sq_smem_u32(smem) + (wsb >> 1) * SQ_BOX_BYTES + lm_row * 128;   // box wsb / 2
    const uint32_t x_cb = static_cast<uint32_t>((4 * (wsb & 1)) << 4);                       // first chunk of super-block wsb in its box row
    // (super-block q, k-step ks) -> chunk c = 4q + 2ks (+1 for lanes >= 16), at byte ((c ^ (row & 7)) << 4):
    // x_sw holds the lane's XOR term, already shifted
    // (g = 16: the lane's chunks are tig and 4 + tig of its own row, XOR term prow & 7)
    const uint32_t x_sw = LDSM ? static_cast<uint32_t>(((lane >> 4) ^ (lane & 7)) << 4)
                               : static_cast<uint32_t>((tig ^ (prow & 7)) << 4);
    // (the host takes this kernel only while both output buffers stay below 4 GiB: 32-bit byte offsets)
    const uint32_t code_pitch32 = static_cast<uint32_t>(code_pitch);
    const uint32_t code_step = SQ_ROWS * code_pitch32;
    const bool m_ragged = (M % SQ_ROWS) != 0;
    uint32_t code_off = 0;                    // codes of (row rA, this lane's 8 bytes) for the current item
    for (int it = item_begin; it < item_end; ++it, ++n) {
      const int nsb = min(4, total_sb - panel * 4);
      if (panel != cur_panel) {
        cur_panel = panel;
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
          const int sb = panel * 4 + wsb + q;
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            const int r = 8 * nchunk + 2 * t + (gid & 1);     // transform row for column slot gid of tile t
            // B fragment of column slot gid: channels 2*tig, 2*tig+1 (+8) of k-step 0 in .x (.y), of k-step 1 in .z (.w)
            if (NSPLIT == 1) {
              uint4 w = make_uint4(0, 0, 0, 0);
              if (wsb + q < nsb) {
                if (G == 32) {
                  const uint32_t* row = reinterpret_cast<const uint32_t*>(T + ((int64_t)sb * 32 + r) * 32);
                  w = make_uint4(__ldg(row + tig), __ldg(row + 4 + tig), __ldg(row + 8 + tig), __ldg(row + 12 + tig));
                } else if ((r >> 4) == (tig >> 1)) {
                  // permuted contraction index: the lane's 8 channels 8*tig.. belong to block tig >> 1 of the
                  // block-diagonal pair; off-diagonal pieces are zero
                  w = __ldg(reinterpret_cast<const uint4*>(T + (((int64_t)sb * 2 + (r >> 4)) * 16 + (r & 15)) * 16 + 8 * (tig & 1)));
                }
              }
              tf[0][q][t] = w;
            } else {
              // the same eight entries as above, from the fp32 matrix, each split into hi + mid + lo
              float f[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) f[i] = 0.f;
              if (wsb + q < nsb) {
                if (G == 32) {
                  const float2* row = reinterpret_cast<const float2*>(Tf + ((int64_t)sb * 32 + r) * 32);
#pragma unroll
                  for (int i = 0; i < 4; ++i) { const float2 v = __ldg(row + 4 * i + tig); f[2 * i] = v.x; f[2 * i + 1] = v.y; }
                } else if ((r >> 4) == (tig >> 1)) {
                  const float4* row = reinterpret_cast<const float4*>(Tf + (((int64_t)sb * 2 + (r >> 4)) * 16 + (r & 15)) * 16 + 8 * (tig & 1));
                  const float4 v0 = __ldg(row), v1 = __ldg(row + 1);
                  f[0] = v0.x; f[1] = v0.y; f[2] = v0.z; f[3] = v0.w; f[4] = v1.x; f[5] = v1.y; f[6] = v1.z; f[7] = v1.w;
                }
              }
              uint32_t pk[3][4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                __nv_bfloat16 h[2][3];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                  const float x = f[2 * i + e];
                  h[e][2] = __float2bfloat16_rn(x);
                  const float r1 = x - __bfloat162float(h[e][2]);               // exact
                  h[e][1] = __float2bfloat16_rn(r1);
                  const float r2 = r1 - __bfloat162float(h[e][1]);              // exact
                  h[e][0] = __float2bfloat16_rn(r2);
                }
#pragma unroll
                for (int sp = 0; sp < 3; ++sp)
                  pk[sp][i] = (uint32_t)__bfloat16_as_ushort(h[0][sp]) | ((uint32_t)__bfloat16_as_ushort(h[1][sp]) << 16);
              }
#pragma unroll
              for (int sp = 0; sp < NSPLIT; ++sp) tf[sp][q][t] = make_uint4(pk[sp][0], pk[sp][1], pk[sp][2], pk[sp][3]);
            }
          }
        }
        // output pointers of this panel at the current row block
        const uint32_t rA0 = rb * SQ_ROWS + prow;
        // NQ = 2: after the exchange below lane tig owns bytes 8 tig .. 8 tig + 7 of the pair's 32;  NQ = 1: the
        // lane's 8 outputs are transform rows 8 c .. 8 c + 7, c = (0,2,1,3)[tig], i.e. bytes 4 c .. 4 c + 3 of 16
        code_off = rA0 * code_pitch32 + (panel * 64 + wsb * 16 + (NQ == 2 ? 8 * tig : 4 * (((tig & 1) << 1) | (tig >> 1))));
      }
      const int s = n % SQ_STAGES;
      const uint32_t ph = (n / SQ_STAGES) & 1;
      if (!__all_sync(0xffffffffu, sq_wait(sq_smem_u32(&full_bar[s]), ph, abort_flag))) {
        if (lane == 0) { if (*abort_flag == 0 && status) atomicExch(status, 0x50000 | n); *abort_flag = 1; }
        break;
      }
      uint4 af[NQ][2];                          // A operand quads: [super-block q][k-step]
      {
        const uint32_t a = x_base + s * SQ_STAGE_BYTES;
        // chunk index c of a box row sits at byte ((c ^ (row & 7)) << 4).  The chunk bases used here are even
        // (or multiples of 4) and the lane's own term (lane >> 4, or tig) only touches the bits below, so
        // (base + term) ^ r7 = base ^ (term ^ r7): XOR the shifted base with the lane's precomputed x_sw
#pragma unroll
        for (int q = 0; q < NQ; ++q) {          // super-block wsb + q starts at chunk x_cb / 16 + 4 q of its box row
          const uint32_t cb = x_cb + ((4u * q) << 4);
          if (LDSM) {
            af[q][0] = sq_ldmatrix_x4(a + (cb ^ x_sw));
            af[q][1] = sq_ldmatrix_x4(a + ((cb + (2u << 4)) ^ x_sw));
          } else {                              // rows prow and prow + 8 share the XOR term; the lane's chunk is cb / 16 + tig
            const uint4 xa = sq_lds128(a + (cb ^ x_sw)), xb = sq_lds128(a + (cb ^ x_sw) + 8 * 128);
            af[q][0] = make_uint4(xa.x, xb.x, xa.y, xb.y);
            af[q][1] = make_uint4(xa.z, xb.z, xa.w, xb.w);
          }
        }
      }
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(sq_smem_u32(&empty_bar[s])) : "memory");

      uint8_t* const pa = codes + code_off;
      uint8_t* ps;                              // scale byte of (row rA, first block of this warp's first super-block)
      {
        const uint32_t rA0 = rb * SQ_ROWS + prow;
        const int kb0 = (G == 32) ? cur_panel * 4 + wsb : cur_panel * 8 + 2 * wsb;
        if (sf_layout == 0) ps = scales + (rA0 * KB32 + kb0);
        else ps = scales + (((rA0 >> 7) * ktiles + (kb0 >> 2)) * 512 + (rA0 & 31) * 16 + ((rA0 & 127) >> 5) * 4 + (kb0 & 3));
      }
      const int this_rb = rb;
      const bool last_rb = (rb == num_rb - 1);
      if (++rb == num_rb) { rb = 0; ++panel; } else { code_off += code_step; }
      if (wsb >= nsb) continue;                 // K tail: this warp's super-blocks do not exist

      // One item: FULL = every row and both super-blocks of this warp exist (no predicates at all).
      auto item = [&](auto full_tag) {
        constexpr bool FULL = decltype(full_tag)::value;
        bool okA = true, okB = true;
        if (!FULL) {
          const int rA = this_rb * SQ_ROWS + prow;                       // only the last row block can be ragged
          okA = !last_rb || rA < M;
          okB = !last_rb || rA + 8 < M;
        }
        uint32_t wA[NQ], wB[NQ], sA[NQ], sB[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
          float acc[4][4];
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            mma_bf16_16816_first(acc[t], af[q][0].x, af[q][0].y, af[q][0].z, af[q][0].w, tf[0][q][t].x, tf[0][q][t].y);
            mma_bf16_16816(acc[t], af[q][1].x, af[q][1].y, af[q][1].z, af[q][1].w, tf[0][q][t].z, tf[0][q][t].w);
#pragma unroll
            for (int sp = 1; sp < NSPLIT; ++sp) {
              mma_bf16_16816(acc[t], af[q][0].x, af[q][0].y, af[q][0].z, af[q][0].w, tf[sp][q][t].x, tf[sp][q][t].y);
              mma_bf16_16816(acc[t], af[q][1].x, af[q][1].y, af[q][1].z, af[q][1].w, tf[sp][q][t].z, tf[sp][q][t].w);
            }
          }
          float vA[8], vB[8];
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            vA[2 * t] = acc[t][0]; vA[2 * t + 1] = acc[t][1];
            vB[2 * t] = acc[t][2]; vB[2 * t + 1] = acc[t][3];
          }
          // AbsMax of the lane's 8 values per row as a tree of 3-input maxima (sm_100 has a 3-input FMNMX)
          float aA = fmaxf(fmaxf(fabsf(vA[0]), fabsf(vA[1])), fabsf(vA[2]));
          aA = fmaxf(fmaxf(aA, fabsf(vA[3])), fabsf(vA[4]));
          aA = fmaxf(fmaxf(aA, fabsf(vA[5])), fmaxf(fabsf(vA[6]), fabsf(vA[7])));
          float aB = fmaxf(fmaxf(fabsf(vB[0]), fabsf(vB[1])), fabsf(vB[2]));
          aB = fmaxf(fmaxf(aB, fabsf(vB[3])), fabsf(vB[4]));
          aB = fmaxf(fmaxf(aB, fabsf(vB[5])), fmaxf(fabsf(vB[6]), fabsf(vB[7])));
          if (AMAX) { seen = fmaxf(seen, fmaxf(okA ? aA : 0.0f, okB ? aB : 0.0f)); continue; }
          aA = fmaxf(aA, __shfl_xor_sync(0xffffffffu, aA, 2));       // lanes tig and tig^2 share a g=16 block
          aB = fmaxf(aB, __shfl_xor_sync(0xffffffffu, aB, 2));
          if (G == 32) {
            aA = fmaxf(aA, __shfl_xor_sync(0xffffffffu, aA, 1));
            aB = fmaxf(aB, __shfl_xor_sync(0xffffffffu, aB, 1));
          }
          float mA, mB;
          if (FMT == kFmtMX) {
            mx_scale(aA, sA[q], mA, mx_ceil); mx_scale(aB, sB[q], mB, mx_ceil);
          } else {
            // four distinct scales per quad (row A/B x block 0/1): lane tig computes the one of
            // (row tig>>1, its own block) and fetches the other row's from lane tig^2
            const bool mine_is_b = (tig >> 1) != 0;
            const uint32_t sm = nv_scale_byte(mine_is_b ? aB : aA, nvf);
            const uint32_t so = __shfl_xor_sync(0xffffffffu, sm, 2);
            sA[q] = mine_is_b ? so : sm; mA = sq_lds_f32(nv_mult_u32 + 4 * sA[q]);
            sB[q] = mine_is_b ? sm : so; mB = sq_lds_f32(nv_mult_u32 + 4 * sB[q]);
          }
          const uint64_t mA2 = pair_of(mA), mB2 = pair_of(mB);       // {m, m} built once per row
#pragma unroll
          for (int i = 0; i < 8; i += 2) { mul2_rn(vA[i], vA[i + 1], mA2); mul2_rn(vB[i], vB[i + 1], mB2); }
          wA[q] = pack_e2m1x8_fast(vA);
          wB[q] = pack_e2m1x8_fast(vB);
        }
        if (AMAX) return;
        const uint32_t sf_row8 = (sf_layout == 0) ? 8 * KB32 : 8 * 16;   // rows rA and rA + 8: same 32-row group of a scale tile
        if (NQ == 2) {
          // ---- codes: lanes 0,1 gather super-block 0, lanes 2,3 super-block 1 (8 contiguous bytes each)
          const bool lo = tig < 2;
          const uint32_t rcvA = __shfl_xor_sync(0xffffffffu, lo ? wA[NQ - 1] : wA[0], 2);
          const uint32_t rcvB = __shfl_xor_sync(0xffffffffu, lo ? wB[NQ - 1] : wB[0], 2);
          const uint2 oA = lo ? make_uint2(wA[0], rcvA) : make_uint2(rcvA, wA[NQ - 1]);
          const uint2 oB = lo ? make_uint2(wB[0], rcvB) : make_uint2(rcvB, wB[NQ - 1]);
          const bool col_ok = FULL || (wsb + (tig >> 1)) < nsb;
          if (okA && col_ok) *reinterpret_cast<uint2*>(pa) = oA;
          if (okB && col_ok) *reinterpret_cast<uint2*>(pa + 8 * code_pitch32) = oB;
          // ---- scale bytes of the pair of super-blocks
          const bool pair_ok = FULL || (wsb + 1 < nsb);
          if (G == 32) {
            if (tig == 0) {                      // one 16-bit store per row
              const uint32_t outA = sA[0] | (sA[NQ - 1] << 8), outB = sB[0] | (sB[NQ - 1] << 8);
              if (pair_ok) {
                if (okA) *reinterpret_cast<uint16_t*>(ps) = (uint16_t)outA;
                if (okB) *reinterpret_cast<uint16_t*>(ps + sf_row8) = (uint16_t)outB;
              } else {
                if (okA) ps[0] = (uint8_t)outA;
                if (okB) ps[sf_row8] = (uint8_t)outB;
              }
            }
          } else {
            // lanes tig 0,2 hold the first block of each super-block, lanes 1,3 the second: one 32-bit store per row
            const uint32_t mineA = sA[0] | (sA[NQ - 1] << 16), mineB = sB[0] | (sB[NQ - 1] << 16);
            const uint32_t othA = __shfl_xor_sync(0xffffffffu, mineA, 1), othB = __shfl_xor_sync(0xffffffffu, mineB, 1);
            if (tig == 0) {
              const uint32_t outA = mineA | (othA << 8), outB = mineB | (othB << 8);
              if (pair_ok) {
                if (okA) *reinterpret_cast<uint32_t*>(ps) = outA;
                if (okB) *reinterpret_cast<uint32_t*>(ps + sf_row8) = outB;
              } else {
                if (okA) *reinterpret_cast<uint16_t*>(ps) = (uint16_t)outA;
                if (okB) *reinterpret_cast<uint16_t*>(ps + sf_row8) = (uint16_t)outB;
              }
            }
          }
        } else {
          // ---- one super-block per warp: every lane stores its own 4 code bytes (a quad covers the 16 bytes)
          if (okA) *reinterpret_cast<uint32_t*>(pa) = wA[0];
          if (okB) *reinterpret_cast<uint32_t*>(pa + 8 * code_pitch32) = wB[0];
          if (G == 32) {
            if (tig == 0) {
              if (okA) ps[0] = (uint8_t)sA[0];
              if (okB) ps[sf_row8] = (uint8_t)sB[0];
            }
          } else {                               // the super-block's two block scales: lanes tig 0 and 1
            const uint32_t othA = __shfl_xor_sync(0xffffffffu, sA[0], 1), othB = __shfl_xor_sync(0xffffffffu, sB[0], 1);
            if (tig == 0) {
              if (okA) *reinterpret_cast<uint16_t*>(ps) = (uint16_t)(sA[0] | (othA << 8));
              if (okB) *reinterpret_cast<uint16_t*>(ps + sf_row8) = (uint16_t)(sB[0] | (othB << 8));
            }
          }
        }
      };
      if (nsb == 4 && !(last_rb && m_ragged)) item(std::true_type());
      else item(std::false_type());
    }
    if (AMAX) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) seen = fmaxf(seen, __shfl_xor_sync(0xffffffffu, seen, o));
      if (lane == 0 && ts_out != nullptr) atomicMax(reinterpret_cast<uint32_t*>(ts_out), __float_as_uint(seen));
    }
  }
  __syncthreads();
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*SqEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                               const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static SqEncodeFn sq_encode_fn() {
  static SqEncodeFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<SqEncodeFn>(p);
  }
  return fn;
}

// One launch for a given tile height.  cudaErrorNotSupported: use the register-staged kernel instead.
template <int ROWS, int NSPLIT = 1>
static cudaError_t launch_stream(const void* X, int64_t M, int64_t K, const void* T, int g, const float* ts,
                                 uint8_t* codes, uint8_t* scales, int sf, int32_t* status, bool clear_status, bool pdl,
                                 cudaStream_t st, const QuantOpts& opt, int sm_count) {
  SqEncodeFn enc = sq_encode_fn();
  CUtensorMap map;
  const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)ROWS};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(X), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorNotSupported;
  static bool attr_done_of[kDeviceSlots] = {};
  const int slot = device_slot();
  if (slot < 0) return cudaErrorInvalidDevice;
  bool& attr_done = attr_done_of[slot];
  cudaError_t e;
  if (!attr_done) {
    if ((e = cudaFuncSetAttribute(tq_stream_kernel<32, false, ROWS, NSPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SQ_SMEM)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(tq_stream_kernel<16, false, ROWS, NSPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SQ_SMEM)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(tq_stream_kernel<16, true, ROWS, NSPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SQ_SMEM)) != cudaSuccess) return e;
    attr_done = true;
  }
  const int num_rb = (int)((M + ROWS - 1) / ROWS);
  const int64_t panels = (K / 32 + 3) / 4;
  const int64_t items = panels * num_rb;
  if (items > 0x7fffffff || M > 0x7fffff00) return cudaErrorNotSupported;
  if ((M + ROWS) * (K / 2) >= ((int64_t)1 << 32)) return cudaErrorNotSupported;   // the kernel keeps 32-bit output offsets
  const int grid = (int)(items < sm_count ? items : sm_count);
  const void* Tb = T;
  const int cs = clear_status ? 1 : 0;
  const int n_items = (int)items;
  const uint32_t* amax_in = opt.amax_in;
  float* ts_out = opt.ts_out;
  const int mx_ceil = opt.mx_ceil ? 1 : 0;
  const int drop = opt.drop_item;
  if (opt.amax_out != nullptr) {                 // AbsMax pass only (g = 16)
    if (g != 16) return cudaErrorNotSupported;
    tq_stream_kernel<16, true, ROWS, NSPLIT><<<grid, SQ_THREADS, SQ_SMEM, st>>>(map, Tb, M, K, nullptr, nullptr, nullptr, sf, num_rb, n_items,
                                                                        status, cs, nullptr, reinterpret_cast<float*>(opt.amax_out), 0, -1);
    return cudaGetLastError();
  }
  if (!pdl) {
    if (g == 32)
      tq_stream_kernel<32, false, ROWS, NSPLIT><<<grid, SQ_THREADS, SQ_SMEM, st>>>(map, Tb, M, K, ts, codes, scales, sf, num_rb, n_items, status, cs, amax_in, ts_out, mx_ceil, drop);
    else
      tq_stream_kernel<16, false, ROWS, NSPLIT><<<grid, SQ_THREADS, SQ_SMEM, st>>>(map, Tb, M, K, ts, codes, scales, sf, num_rb, n_items, status, cs, amax_in, ts_out, mx_ceil, drop);
    return cudaGetLastError();
  }
  // programmatic dependent launch: set-up overlaps the tail of the previous kernel of the stream
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(SQ_THREADS, 1, 1);
  cfg.dynamicSmemBytes = SQ_SMEM;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (g == 32)
    return cudaLaunchKernelEx(&cfg, tq_stream_kernel<32, false, ROWS, NSPLIT>, map, Tb, M, K, ts, codes, scales, sf, num_rb, n_items, status, cs, amax_in, ts_out, mx_ceil, drop);
  return cudaLaunchKernelEx(&cfg, tq_stream_kernel<16, false, ROWS, NSPLIT>, map, Tb, M, K, ts, codes, scales, sf, num_rb, n_items, status, cs, amax_in, ts_out, mx_ceil, drop);
}

static cudaError_t stream_sm_count(int* out) {
  static int sm_count_of[kDeviceSlots] = {};
  const int slot = device_slot();
  if (slot < 0) return cudaErrorInvalidDevice;
  if (sm_count_of[slot] == 0) {
    int sms = 0;
    const cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, slot);
    if (e != cudaSuccess) return e;
    sm_count_of[slot] = sms;
  }
  *out = sm_count_of[slot];
  return cudaSuccess;
}

// Weight side through the same kernel: W[N,K] bf16, Tinv fp32 (three-way split), 64-row tiles.  opt carries
// the AbsMax pass / tensor-scale pointers for NVFP4 exactly as on the activation side.
cudaError_t run_quantize_weight_stream(const void* W, int64_t N, int64_t K, const float* Tinv, int g, uint8_t* codes,
                                       uint8_t* scales, int sf, cudaStream_t st, const QuantOpts& opt) {
  if (opt.force_rows == 0 && N > 256) {          // first choice: the tcgen05 kernel (as on the activation side)
    const cudaError_t et = run_quantize_weight_tc(W, N, K, Tinv, g, codes, scales, sf, st, opt);
    if (et != cudaErrorNotSupported) return et;
  }
  if (!sq_encode_fn()) return cudaErrorNotSupported;
  if (sf == 0 && ((K / g) & 3) != 0) return cudaErrorNotSupported;
  int sm_count = 0;
  const cudaError_t e = stream_sm_count(&sm_count);
  if (e != cudaSuccess) return e;
  return launch_stream<64, 3>(W, N, K, Tinv, g, nullptr, codes, scales, sf, nullptr, false, false, st, opt, sm_count);
}

// Returns cudaErrorNotSupported when the streaming kernel cannot take the problem (the caller
// then uses the register-staged kernel).
cudaError_t run_quantize_act_stream(const void* X, int64_t M, int64_t K, const void* T, int g, const float* ts,
                                    uint8_t* codes, uint8_t* scales, int sf, int32_t* status, bool clear_status, bool pdl,
                                    cudaStream_t st, const QuantOpts& opt) {
  // First choice: the kernel that runs the block products on the tcgen05 tensor cores.  The warp-level kernel below
  // remains for the weight side (fp32 transforms, three-way split), as the fall-back, and under the test hook that
  // forces one of its tile heights.
  // (decode-sized batches stay on the warp-level kernel: a launch with a handful of 128-row items is dominated by
  // set-up, and that kernel has 1-2 us less of it - no tensor-memory allocation, a third of the threads)
  if (opt.force_rows == 0 && M > 256) {
    const cudaError_t et = run_quantize_act_tc(X, M, K, T, g, ts, codes, scales, sf, status, clear_status, pdl, st, opt);
    if (et != cudaErrorNotSupported) return et;
  }
  if (!sq_encode_fn()) return cudaErrorNotSupported;
  if (sf == 0 && ((K / g) & 3) != 0) return cudaErrorNotSupported;      // LINEAR rows must keep 4-byte scale groups aligned
  int sm_count = 0;
  const cudaError_t e0 = stream_sm_count(&sm_count);
  if (e0 != cudaSuccess) return e0;
  // 128-row tiles unless the problem is small: with fewer than SQ_SMALL of them per CTA the 64-row tiles'
  // finer items win (the first tile lands sooner and the CTAs finish closer together)
  const int64_t items128 = ((K / 32 + 3) / 4) * ((M + 127) / 128);
  const bool rows64 = opt.force_rows ? (opt.force_rows == 64) : (items128 < (int64_t)SQ_SMALL * sm_count);
  if (rows64)
    return launch_stream<64>(X, M, K, T, g, ts, codes, scales, sf, status, clear_status, pdl, st, opt, sm_count);
  return launch_stream<128>(X, M, K, T, g, ts, codes, scales, sf, status, clear_status, pdl, st, opt, sm_count);
}

}  // namespace wush
