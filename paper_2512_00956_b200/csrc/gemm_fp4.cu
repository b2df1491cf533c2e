// Block-scaled FP4 GEMM on 5th-generation tensor cores (Eq. 7, outer sum):
//   Y[m,n] = alpha * sum_c sx[m,c] sw[n,c] sum_{k in c} xq[m,k] wq[n,k]
// MXFP4 uses tcgen05.mma kind::mxf4 (E8M0 scales, one per 32 elements); NVFP4 uses
// kind::mxf4nvf4 (E4M3 scales, one per 16 elements).  Accumulation is fp32 in tensor memory.
//
// This is the kernel for M <= 128 (decode, small batches), where the layer is bound by streaming
// the weights once from HBM: one CTA computes one 128 x 128 tile of Y, two CTAs share an SM, so
// N/128 CTAs keep every SM pulling weight bytes.  (M > 128 goes to the two-CTA kernel.)
// Warp 0 streams operands: per 256-element K slab two TMA tile loads (128-byte swizzle, K-major
// packed FP4 bytes) and the matching scale tiles (plain bulk copies of the 512-byte GEMM-native
// scale tiles) into a ring of 3 to 5 stages (see stages_of) guarded by full/empty mbarriers.  One thread of warp 1 copies the scale tiles into tensor memory
// (tcgen05.cp) and issues four K=64 MMAs per slab; tcgen05.commit releases the stage.
// Warps 2-5 drain the accumulator (tcgen05.ld), apply alpha and store Y.
//
// Every wait is bounded: if a barrier does not flip within about two seconds the waiting
// role raises a CTA-wide abort flag, writes a diagnostic word to *status, and every role
// falls through to the common exit where in-flight copies are drained and tensor memory is
// released.  No TMA load uses cluster multicast.
#include <cuda.h>

#include "wush_device.cuh"
#include "wush_host.h"

namespace wush {

constexpr int BM = 128;             // tile rows (tokens)
constexpr int BN = 128;             // tile columns (output channels)
constexpr int BKB = 128;            // bytes of packed FP4 per row per stage = 256 elements
constexpr int A_BYTES = BM * BKB;   // 16 KiB: what one MMA reads, whatever part of it the A box fills
constexpr int B_BYTES = BN * BKB;   // 16 KiB
constexpr int GEMM_THREADS = 192;
constexpr uint32_t TMEM_COLS = 256;  // two co-resident CTAs fit in the 512 columns of an SM
constexpr uint32_t SFA_COL = 128;   // tensor-memory column of the A scales (after the 128 accumulator columns)
constexpr uint32_t SFB_COL = 160;   // B scales: 4 columns per scale tile

__host__ __device__ constexpr int sf_tiles_per_stage(int fmt) { return fmt == kFmtMX ? 2 : 4; }
__host__ __device__ constexpr int stage_sf_bytes(int fmt) { return 2 * sf_tiles_per_stage(fmt) * 512; }
// Ring depth.  The kernel is bound by streaming the weights, and what a CTA streams is set by the bytes it has in
// flight (about 2 us from request to arrival under load): with few tokens the activation slot of a stage shrinks
// to the rows that exist (a_rows = 16, 32, 64 or 128) and the ring gets as many stages as still let two CTAs share
// an SM (3 with 128 rows; 5 with 16).  An MMA always reads 128 rows: the rows beyond the slot are whatever follows
// it in the ring (all FP4 bit patterns are finite numbers) and only reach accumulator rows that are never stored.
constexpr int SMEM_PER_CTA = (228 * 1024 - 2 * 1024) / 2;   // two CTAs per SM, 1 KiB reserved for each
__host__ __device__ constexpr int stage_bytes(int fmt, int a_rows) { return a_rows * BKB + B_BYTES + stage_sf_bytes(fmt); }
__host__ __device__ constexpr int stages_of(int fmt, int a_rows) { return (SMEM_PER_CTA - 1024 - 256) / stage_bytes(fmt, a_rows); }
__host__ __device__ constexpr int gemm_smem_bytes(int fmt, int a_rows) {
  // alignment slack + ring + barriers; the last activation slot is read 16 KiB deep, so with short slots the
  // weight slots that follow it must exist: they do, the ring is laid out [A slots][B slots][scale tiles]
  return 1024 + stages_of(fmt, a_rows) * stage_bytes(fmt, a_rows) + 256;
}
static_assert(stages_of(kFmtMX, 128) == 3 && stages_of(kFmtNV, 128) == 3 && stages_of(kFmtMX, 16) == 5 && stages_of(kFmtNV, 16) == 5, "ring depth");

// ------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: false if the phase did not complete within ~2 s or another role aborted.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < 4096; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  while (true) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag != 0) return false;
    if (global_timer_ns() - t0 > 2000000000ull) return false;
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
// true in exactly one lane of a fully converged warp
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_cp_sf(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
template <int FMT>
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t sfa, uint32_t sfb, uint32_t accumulate) {
  if (FMT == kFmtMX) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.scale_vec::4X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
        : "memory");
  }
}
__device__ __forceinline__ void tc_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand tile written by TMA with the 128-byte
// swizzle: rows are 128 bytes, groups of 8 rows (1024 bytes) follow each other.
//   bits [0,14)  start address >> 4        bits [32,46) stride between 8-row groups >> 4
//   bits [46,48) descriptor version 1      bits [61,64) swizzle mode (2 = 128 B)
__device__ __forceinline__ uint64_t operand_desc(uint32_t smem_addr) {
  return static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) /* leading offset: unused, 1 */ |
         (static_cast<uint64_t>(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Descriptor of a 512-byte scale tile (32 rows x 16 bytes, no swizzle; 8-row core matrices of
// 128 bytes stacked along the row axis).
__device__ __forceinline__ uint64_t scale_desc(uint32_t smem_addr) {
  return static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(128 >> 4) << 32) |
         (1ull << 46);
}
// Instruction descriptor, block-scaled kinds:  [4,6) B scale byte offset, [7,10) A format and
// [10,13) B format (1 = E2M1), [15]/[16] A/B major (0 = K), [17,23) N/8, [23] scale type
// (0 = E4M3, 1 = E8M0), [24,29) M/16, [29,31) A scale byte offset, [31] K size (0 = 64).
__device__ __forceinline__ uint32_t instr_desc(int fmt, uint32_t sf_byte) {
  return (sf_byte << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
         ((fmt == kFmtMX ? 1u : 0u) << 23) | (static_cast<uint32_t>(BM >> 4) << 24) | (sf_byte << 29);
}

// ------------------------------------------------------------------------------ the kernel
template <int FMT, int A_ROWS>
__global__ void __launch_bounds__(GEMM_THREADS, 2)
gemm_fp4_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                const uint8_t* __restrict__ SFA, const uint8_t* __restrict__ SFB, int M, int N, int K,
                const float* __restrict__ tsx, const float* __restrict__ tsw, void* __restrict__ Yout,
                int out_bf16, int32_t* __restrict__ status, int a_box_bytes, int clear_status) {
  constexpr int TPS = sf_tiles_per_stage(FMT);           // scale tiles (4 scale columns each) per stage
  constexpr int KSTEPS_PER_TILE = (FMT == kFmtMX) ? 2 : 1;  // K=64 MMAs covered by one scale tile
  constexpr int STAGES = stages_of(FMT, A_ROWS);
  constexpr int A_SLOT = A_ROWS * BKB;                   // bytes between the activation slots of consecutive stages
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = sA + STAGES * A_SLOT;
  uint8_t* sSF = sB + STAGES * B_BYTES;                   // per stage: [A tiles][B tiles]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sSF + STAGES * stage_sf_bytes(FMT));
  uint64_t* full_bar = bars;
  uint64_t* empty_bar = bars + STAGES;
  uint64_t* tmem_full_bar = bars + 2 * STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * BN, m0 = blockIdx.y * BM;
  const int num_kb = (K + 2 * BKB - 1) / (2 * BKB);       // 256-element slabs
  const int sf_cols = K / (FMT == kFmtMX ? 32 : 16);
  const int ktiles_total = (sf_cols + 3) >> 2;            // scale tiles along K

  if (threadIdx.x == 64) { prefetch_tensormap(&mapB); prefetch_tensormap(&mapA); }
  // stand-alone call: the first CTA clears the status word (a report can only follow a wait of about two
  // seconds, so this cannot erase one); inside wush_linear the quantiser kernel has cleared it
  if (clear_status && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 96 && status != nullptr) *status = 0;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
    mbar_init(smem_u32(tmem_full_bar), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // see the two-CTA kernel

  if (warp == 0) {
    // ------------------------------------------------------------------ operand producer
    // The whole warp walks the loop (warp-uniform control flow keeps addresses and descriptors in
    // uniform registers); one elected lane issues the copies.
    int issued = 0;
    bool ok = true;
    // Weights do not depend on the preceding kernel of the stream.  Launched as a programmatic dependent of
    // the quantiser, this CTA may start while that kernel still runs: the first ring-full of weight tiles and
    // weight scales is requested at once, the activation side only after the quantiser has completed.
    // (The whole stage's byte count is announced with the first half, so the barrier flips when both landed.)
    const int pre = min(STAGES, num_kb);
    auto weights = [&](int kb, int s, uint32_t bar, uint32_t sf_bytes) {
      uint8_t* sf = sSF + s * stage_sf_bytes(FMT);
      mbar_expect_tx(bar, a_box_bytes + B_BYTES + sf_bytes * 2);
      tma_load_2d(smem_u32(sB + s * B_BYTES), &mapB, kb * BKB, n0, bar);
      bulk_load_1d(smem_u32(sf + TPS * 512), SFB + ((int64_t)(n0 >> 7) * ktiles_total + kb * TPS) * 512, sf_bytes, bar);
    };
    auto activations = [&](int kb, int s, uint32_t bar, uint32_t sf_bytes) {
      // the A box covers only round_up(M, 8) rows when M < 128: the rows of the stage below it keep stale
      // bytes, which only reach accumulator rows that are never stored
      uint8_t* sf = sSF + s * stage_sf_bytes(FMT);
      tma_load_2d(smem_u32(sA + s * A_SLOT), &mapA, kb * BKB, m0, bar);
      bulk_load_1d(smem_u32(sf), SFA + ((int64_t)(m0 >> 7) * ktiles_total + kb * TPS) * 512, sf_bytes, bar);
    };
    if (elect_one())
      for (int kb = 0; kb < pre; ++kb)
        weights(kb, kb, smem_u32(&full_bar[kb]), min(TPS, ktiles_total - kb * TPS) * 512);
    __syncwarp();
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (elect_one())
      for (int kb = 0; kb < pre; ++kb)
        activations(kb, kb, smem_u32(&full_bar[kb]), min(TPS, ktiles_total - kb * TPS) * 512);
    __syncwarp();
    issued = pre;
    for (int kb = pre; kb < num_kb; ++kb) {
      const int s = kb % STAGES;
      const uint32_t ph = (kb / STAGES) & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1, abort_flag))) {
        if (lane == 0) {
          if (*abort_flag == 0 && status) atomicExch(status, 0x10000 | kb);
          *abort_flag = 1;
        }
        ok = false;
        break;
      }
      const uint32_t sf_bytes = min(TPS, ktiles_total - kb * TPS) * 512;
      const uint32_t bar = smem_u32(&full_bar[s]);
      if (elect_one()) {
        weights(kb, s, bar, sf_bytes);
        activations(kb, s, bar, sf_bytes);
      }
      __syncwarp();
      ++issued;
    }
    if (!ok) {
      // drain: every stage filled must land before the CTA may exit
      for (int kb = max(0, issued - STAGES); kb < issued; ++kb) {
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&full_bar[kb % STAGES]), (kb / STAGES) & 1))
          if (global_timer_ns() - t0 > 500000000ull) break;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    bool ok = true;
    for (int kb = 0; kb < num_kb; ++kb) {
      const int s = kb % STAGES;
      const uint32_t ph = (kb / STAGES) & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&full_bar[s]), ph, abort_flag))) {
        if (lane == 0) {
          if (*abort_flag == 0 && status) atomicExch(status, 0x20000 | kb);
          *abort_flag = 1;
        }
        ok = false;
        break;
      }
      tc_fence_after();
      const int tiles = min(TPS, ktiles_total - kb * TPS);
      const uint32_t sf = smem_u32(sSF + s * stage_sf_bytes(FMT));
      const int ksteps = min(4, (K - kb * 2 * BKB) / 64);
      const uint64_t adesc = operand_desc(smem_u32(sA + s * A_SLOT));
      const uint64_t bdesc = operand_desc(smem_u32(sB + s * B_BYTES));
      if (elect_one()) {
        for (int i = 0; i < tiles; ++i) {
          tc_cp_sf(tmem_base + SFA_COL + 4 * i, scale_desc(sf + i * 512));
          tc_cp_sf(tmem_base + SFB_COL + 4 * i, scale_desc(sf + (TPS + i) * 512));
        }
        for (int j = 0; j < ksteps; ++j) {
          const int tile = j / KSTEPS_PER_TILE;
          const uint32_t sf_byte = (FMT == kFmtMX) ? 2u * (j % KSTEPS_PER_TILE) : 0u;
          tc_mma<FMT>(tmem_base, adesc + 2 * j, bdesc + 2 * j, instr_desc(FMT, sf_byte),
                      tmem_base + SFA_COL + 4 * tile, tmem_base + SFB_COL + 4 * tile, (kb | j) != 0);
        }
        tc_commit(smem_u32(&empty_bar[s]));
      }
      __syncwarp();
    }
    if (elect_one()) tc_commit(smem_u32(tmem_full_bar));
    __syncwarp();
    if (!ok) {   // let outstanding MMAs finish before tensor memory is released
      const uint64_t t0 = global_timer_ns();
      while (!mbar_try_wait(smem_u32(tmem_full_bar), 0))
        if (global_timer_ns() - t0 > 500000000ull) break;
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;                                 // tensor-memory lane quarter this warp may read
    const int row = m0 + q * 32 + lane;
    bool ok = mbar_wait(smem_u32(tmem_full_bar), 0, abort_flag);
    if (!ok && lane == 0) {
      if (*abort_flag == 0 && status) atomicExch(status, 0x30000 | warp);
      *abort_flag = 1;
    }
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0 && (*abort_flag == 0);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      // *tsx may have been written by the preceding kernel of the stream (per-batch tensor scale); as a
      // programmatic dependent this grid may read it only after that kernel has completed
      asm volatile("griddepcontrol.wait;" ::: "memory");
      float alpha = 1.0f;
      if (FMT == kFmtNV) alpha = __fmul_rn(*tsx, *tsw);
      for (int c = 0; c < BN / 32; ++c) {
        const int col = n0 + c * 32;
        if (col >= N) break;                                // warp-uniform
        uint32_t r[32];
        tc_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + c * 32, r);
        tc_wait_ld();
        if (row < M) {
          if (out_bf16) {
            __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(Yout) + (int64_t)row * N + col;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (col + 8 * v < N) {
                uint32_t p[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[8 * v + 2 * e]) * alpha,
                                                           __uint_as_float(r[8 * v + 2 * e + 1]) * alpha);
                  p[e] = *reinterpret_cast<uint32_t*>(&h);
                }
                *reinterpret_cast<uint4*>(y + 8 * v) = make_uint4(p[0], p[1], p[2], p[3]);
              }
            }
          } else {
            float* y = reinterpret_cast<float*>(Yout) + (int64_t)row * N + col;
#pragma unroll
            for (int v = 0; v < 8; ++v) {
              if (col + 4 * v < N)
                *reinterpret_cast<float4*>(y + 4 * v) =
                    make_float4(__uint_as_float(r[4 * v]) * alpha, __uint_as_float(r[4 * v + 1]) * alpha,
                                __uint_as_float(r[4 * v + 2]) * alpha, __uint_as_float(r[4 * v + 3]) * alpha);
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Tensor map over a row-major [rows][row_bytes] byte matrix, box = 128 bytes x box_rows.
static bool make_operand_map(CUtensorMap* map, const void* base, int64_t rows, int64_t row_bytes, int box_rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
  const cuuint32_t box[2] = {(cuuint32_t)BKB, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t run_gemm_fp4(const uint8_t* Xq, const uint8_t* Xs, const uint8_t* Wq, const uint8_t* Ws,
                         int64_t M, int64_t N, int64_t K, int fmt, const float* tsx, const float* tsw,
                         void* Y, int out_bf16, int32_t* status, bool clear_status, bool after_quantizer, cudaStream_t st,
                         const char** why) {
  cudaError_t e;
  const int cs = (status && clear_status) ? 1 : 0;
  if (M > 128) {
    e = run_gemm_fp4_2cta(Xq, Xs, Wq, Ws, M, N, K, fmt, tsx, tsw, Y, out_bf16, status, cs != 0, after_quantizer, st);
    if (e != cudaErrorNotSupported) return e;
  }
  CUtensorMap mapA, mapB;
  const int a_rows = M >= BM ? BM : (int)((M + 7) / 8 * 8);
  if (!make_operand_map(&mapA, Xq, M, K / 2, a_rows) || !make_operand_map(&mapB, Wq, N, K / 2, BN)) {
    if (why) *why = "cuTensorMapEncodeTiled unavailable or rejected the operand layout";
    return cudaErrorInvalidValue;
  }
  dim3 grid((unsigned)((N + BN - 1) / BN), (unsigned)((M + BM - 1) / BM));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = after_quantizer ? 1 : 0;          // programmatic dependent of the quantiser inside wush_linear
  const int mi = (int)M, ni = (int)N, ki = (int)K, a_bytes = a_rows * BKB;
  const int slot_rows = a_rows <= 16 ? 16 : a_rows <= 32 ? 32 : a_rows <= 64 ? 64 : 128;
  auto go = [&](auto kernel, int smem, bool* attr_done) -> cudaError_t {
    const int slot = device_slot();
    if (slot < 0) return cudaErrorInvalidDevice;
    if (!attr_done[slot]) {
      const cudaError_t ea = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (ea != cudaSuccess) return ea;
      attr_done[slot] = true;
    }
    cfg.dynamicSmemBytes = smem;
    return cudaLaunchKernelEx(&cfg, kernel, mapA, mapB, Xs, Ws, mi, ni, ki, tsx, tsw, Y, out_bf16, status, a_bytes, cs);
  };
#define WUSH_GEMM_CASE(F, R)                                                                  \
  if (fmt == F && slot_rows == R) {                                                           \
    static bool attr_done[kDeviceSlots] = {};                                                 \
    return go(gemm_fp4_kernel<F, R>, gemm_smem_bytes(F, R), attr_done);                       \
  }
  WUSH_GEMM_CASE(kFmtMX, 16) WUSH_GEMM_CASE(kFmtMX, 32) WUSH_GEMM_CASE(kFmtMX, 64) WUSH_GEMM_CASE(kFmtMX, 128)
  WUSH_GEMM_CASE(kFmtNV, 16) WUSH_GEMM_CASE(kFmtNV, 32) WUSH_GEMM_CASE(kFmtNV, 64) WUSH_GEMM_CASE(kFmtNV, 128)
#undef WUSH_GEMM_CASE
  return cudaErrorInvalidValue;
}

}  // namespace wush
