// Fused block transform + quantise (Eq. 7 inner term) with the g x g products on the tcgen05 tensor cores.
//
// Why a second formulation.  The warp-level kernel (transform_quant_stream.cu) spends 120-180 instructions per
// 16 x 32 unit on moving operands into mma.sync fragments, on shuffles between the four lanes that share a block
// and on the MMAs themselves, and ends up half issue-bound.  Here the product is one tcgen05.mma per block
// (A = the 128-row tile of X in shared memory exactly as TMA wrote it, B = the block's transform, D in tensor
// memory), and tcgen05.ld.32x32b hands every thread ONE ROW's outputs of a whole block: AbsMax, scale, rounding and
// packing happen inside a thread, without a single shuffle, and a thread stores its row's 32 code bytes as one
// full sector.  About 35 instructions per unit: the kernel is left with the memory stream.
//
//  * Work item: 128 token rows x 128 channels (two 128-byte-wide TMA boxes, 32 KB; rows are read 256 contiguous
//    bytes at a time).  Items are numbered panel-major (128-channel panel, then row block); a persistent CTA (one
//    per SM) takes a contiguous run.
//  * Ring of 4 stages: 32 KB of X + 2 x 4 KB for the panel's transforms, laid out as B operands, one per box
//    (K-major rows of 128 bytes, 128-byte swizzle: g = 32 -> 32 rows [T_2p[j][0..32) | T_2p+1[j][0..32)],
//    g = 16 -> 16 rows [T_4p[j] | T_4p+1[j] | T_4p+2[j] | T_4p+3[j]]).  The producer warp rewrites a stage's
//    transforms only when the stage last held another panel.
//  * Warp 0: producer (TMA + transform tiles).  Warp 1: allocates tensor memory, issues the MMAs (M = 128,
//    N = g, K = 16 per instruction; block b of a box reads A and B at byte offset b * 2g inside the swizzled
//    rows and writes columns [b*g, b*g + g) of the box's 64 accumulator columns) and commits to the stage's
//    "empty" barrier and the accumulator's "full" barrier.  Warps 2-17: two groups of eight epilogue warps
//    (tensor-memory lane quarter = warp % 4, box = (warp - 2) / 4 % 2); group n % 2 handles item n, so two items
//    are in the epilogue at once.
//  * 4 accumulator buffers of 128 columns = all 512 columns of tensor memory.
//
// Every wait is bounded (about a second); on expiry the role records a diagnostic word, raises the CTA's abort
// flag, every role falls through to the exit, the producer lets requested copies land and tensor memory is freed.
#include <cuda.h>

#include "wush_device.cuh"
#include "wush_host.h"

namespace wush {
namespace tc {

constexpr int ROWS = 128;
constexpr int SUBS = 2;                        // 64-channel boxes per item: rows are read 256 contiguous bytes at a time
constexpr int BOX_BYTES = ROWS * 128;          // 128 rows x 64 bf16 channels
constexpr int X_BYTES = SUBS * BOX_BYTES;
constexpr int TSUB_BYTES = 4096;               // transforms of one 64-channel box as a B operand (one bf16 term)
constexpr int STAGES = 8 / SUBS;
// NSPLIT = 1: bf16 transforms (activations).  NSPLIT = 3: fp32 transforms (weight side) split exactly into three bf16
// terms lo + mid + hi, one B tile each; the three products are accumulated smallest first in the same accumulator.
__host__ __device__ constexpr int t_bytes(int nsplit) { return SUBS * nsplit * TSUB_BYTES; }
__host__ __device__ constexpr int stage_bytes(int nsplit) { return X_BYTES + t_bytes(nsplit); }
constexpr int EPI_WARPS = 16;                  // four groups of four
constexpr int THREADS = (2 + EPI_WARPS) * 32;
constexpr uint32_t TMEM_COLS = 512;
constexpr int ACC_COLS = SUBS * 64;
// ring | full[8] empty[8] tfull[8] tempty[8] (256 B) | tmem slot, abort flag, stage tags (64 B) | NVFP4 multiplier table (512 B)
__host__ __device__ constexpr int smem_bytes(int nsplit) { return 1024 + STAGES * stage_bytes(nsplit) + 256 + 64 + 512; }

__device__ __forceinline__ uint32_t s32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ bool try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t timer_ns() { uint64_t t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
// bounded wait (about one second); false on expiry or when another role has aborted
__device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < 2048; ++i)
    if (try_wait(bar, parity)) return true;
  const uint64_t t0 = timer_ns();
  while (true) {
    for (int i = 0; i < 64; ++i)
      if (try_wait(bar, parity)) return true;
    if (*abort_flag != 0 || timer_ns() - t0 > 1000000000ull) return false;
  }
}
__device__ __forceinline__ bool elect() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[128 x N] (+)= A[128 x 16] B[N x 16]^T, bf16 operands from shared memory, fp32 accumulator in tensor memory
__device__ __forceinline__ void mma_bf16(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ uint64_t op_desc(uint32_t a) {      // K-major, 128-byte swizzle, 8-row groups 1024 B apart
  return static_cast<uint64_t>((a & 0x3FFFFu) >> 4) | (1ull << 16) | (static_cast<uint64_t>(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// kind::f16 instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = 128
__device__ __forceinline__ uint32_t idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(ROWS >> 4) << 24);
}
// 32 consecutive accumulator columns of this thread's tensor-memory lane (valid after tcgen05.wait::ld)
__device__ __forceinline__ void ld32(uint32_t taddr, uint32_t (&u)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]),
        "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]),
        "=r"(u[16]), "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]),
        "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
      : "r"(taddr));
}

// One quantisation block of G values held by one thread: AbsMax, scale byte, multiplier, G/8 packed code words.
// Returns the scale byte.
template <int G>
__device__ __forceinline__ uint32_t quantise_block(const uint32_t* u, int mx_ceil, const NvScaleFast& nvf, uint32_t nv_mult_u32,
                                                   uint32_t* words) {
  // the values are used where tcgen05.ld left them (no copies): AbsMax as two chains of 3-input maxima (sm_100 has a
  // 3-input FMNMX), then packed multiplies into fresh registers that feed the conversions
  auto f = [&](int i) { return __uint_as_float(u[i]); };
  float a0 = fmaxf(fabsf(f(0)), fabsf(f(1))), a1 = fmaxf(fabsf(f(2)), fabsf(f(3)));
#pragma unroll
  for (int i = 4; i < G; i += 4) {
    a0 = fmaxf(fmaxf(a0, fabsf(f(i))), fabsf(f(i + 1)));
    a1 = fmaxf(fmaxf(a1, fabsf(f(i + 2))), fabsf(f(i + 3)));
  }
  const float a = fmaxf(a0, a1);
  uint32_t byte;
  float mult;
  if (G == 32) {
    mx_scale(a, byte, mult, mx_ceil);
  } else {
    byte = nv_scale_byte(a, nvf);
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(mult) : "r"(nv_mult_u32 + 4 * byte));
  }
  const uint64_t mm = pair_of(mult);
#pragma unroll
  for (int w = 0; w < G / 8; ++w) {
    float p[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) mul2_rn_to(p[2 * i], p[2 * i + 1], f(8 * w + 2 * i), f(8 * w + 2 * i + 1), mm);
    words[w] = pack_e2m1x8_fast(p);
  }
  return byte;
}

// The transforms of one 128-channel panel as B operands, one tile per 64-channel box: row j = 128 bytes = the j-th
// rows of the box's 64 / G blocks side by side; 16-byte chunk c of row j sits at chunk c ^ (j & 7) (128-byte swizzle,
// as TMA writes the A operand).  Thread `tid` of `nthreads` copies its share; the caller fences and synchronises.
template <int G, int NSPLIT>
__device__ __forceinline__ void copy_transforms(const void* __restrict__ Tsrc, int panel, int nsub, uint8_t* tdst0, int tid, int nthreads) {
  constexpr int BLOCKS = 64 / G;
  constexpr int CHUNKS = G * 8;                        // 16-byte chunks of a tile: G rows x 8
  constexpr int CPB = G / 8;                           // chunks per block row (64 B or 32 B)
  for (int q = tid; q < nsub * CHUNKS; q += nthreads) {
    const int sub = q / CHUNKS, qq = q % CHUNKS;
    const int j = qq >> 3, c = qq & 7;
    const int blk = (panel * SUBS + sub) * BLOCKS + c / CPB;
    const int64_t src = ((int64_t)blk * G + j) * G + (c % CPB) * 8;           // first of this chunk's 8 entries
    uint8_t* dst = tdst0 + sub * NSPLIT * TSUB_BYTES + j * 128 + ((c ^ (j & 7)) << 4);
    if (NSPLIT == 1) {
      *reinterpret_cast<uint4*>(dst) = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(Tsrc) + src));
    } else {
      const float4* p = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(Tsrc) + src);
      const float4 v0 = __ldg(p), v1 = __ldg(p + 1);
      const float f[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
      uint32_t pk[3][4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint32_t h[2][3];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float x = f[2 * i + e];
          const __nv_bfloat16 hi = __float2bfloat16_rn(x);
          const float r1 = x - __bfloat162float(hi);               // exact
          const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
          const float r2 = r1 - __bfloat162float(mid);              // exact
          const __nv_bfloat16 lo = __float2bfloat16_rn(r2);
          h[e][0] = __bfloat16_as_ushort(lo); h[e][1] = __bfloat16_as_ushort(mid); h[e][2] = __bfloat16_as_ushort(hi);
        }
#pragma unroll
        for (int sp = 0; sp < 3; ++sp) pk[sp][i] = h[0][sp] | (h[1][sp] << 16);
      }
#pragma unroll
      for (int sp = 0; sp < 3; ++sp)                      // tile 0 = lo, 1 = mid, 2 = hi
        *reinterpret_cast<uint4*>(dst + sp * TSUB_BYTES) = make_uint4(pk[sp][0], pk[sp][1], pk[sp][2], pk[sp][3]);
    }
  }
}

// AMAX = true: the same walk and the same products, but only the AbsMax of everything computed is folded into
// *ts_out (bit pattern of a non-negative float, atomicMax): first pass of the per-batch NVFP4 tensor scale.
template <int G, bool AMAX, int NSPLIT = 1>
__global__ void __launch_bounds__(THREADS, 1)
tq_tc_kernel(const __grid_constant__ CUtensorMap mapX, const void* __restrict__ T, int64_t M, int64_t K,
             const float* __restrict__ ts_ptr, uint8_t* __restrict__ codes, uint8_t* __restrict__ scales, int sf_layout,
             int num_panels, int num_items, int32_t* __restrict__ status, int clear_status,
             const uint32_t* __restrict__ amax_in, float* __restrict__ ts_out, int mx_ceil, int drop_item) {
  constexpr int BLOCKS = 64 / G;                     // quantisation blocks per box row: 2 (g = 32) or 4 (g = 16)
  constexpr int STAGE_BYTES = stage_bytes(NSPLIT);
  extern __shared__ uint8_t raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* tfull_bar = empty_bar + STAGES;
  uint64_t* tempty_bar = tfull_bar + STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + STAGES);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* stage_tag = reinterpret_cast<int*>(tmem_slot + 2);                   // panel whose transforms a stage holds
  float* nv_mult = reinterpret_cast<float*>(smem + STAGES * STAGE_BYTES + 256 + 64);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool nv_quant = (G == 16) && !AMAX;
  const bool nv_dynamic = nv_quant && amax_in != nullptr;
  if (threadIdx.x == 32) prefetch_tensormap(&mapX);
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(&full_bar[s])), "r"(2));   // tile requested + transforms in place
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(&empty_bar[s])), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(&tfull_bar[s])), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(&tempty_bar[s])), "r"(4 * SUBS));
      stage_tag[s] = -1;
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  // Launched as a programmatic dependent (wush_linear does), everything above ran while the previous kernel of the
  // stream was still draining; nothing it wrote or still reads may be touched before this point.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (clear_status && blockIdx.x == 0 && threadIdx.x == 0 && status != nullptr) *status = 0;
  float ts = 1.0f;
  if (nv_quant) {                               // tensor scale: possibly the output of the kernel just before this one
    ts = nv_dynamic ? nv_tensor_scale(__uint_as_float(*amax_in)) : *ts_ptr;
    if (threadIdx.x < 128) nv_mult[threadIdx.x] = nv_mult_of_byte(threadIdx.x, ts);
    if (nv_dynamic && blockIdx.x == 0 && threadIdx.x == 0 && ts_out != nullptr) *ts_out = ts;
    __syncthreads();
  }
  // the transforms of the CTA's first STAGES items, copied by all threads at once (later changes of panel - rare, see
  // the grid's size - are the producer warp's job)
  for (int s = 0; s < STAGES; ++s) {
    const int it = blockIdx.x + s * gridDim.x;
    if (it >= num_items) break;
    const int panel = it % num_panels;
    copy_transforms<G, NSPLIT>(T, panel, min(SUBS, (int)(K >> 6) - panel * SUBS), smem + s * STAGE_BYTES + X_BYTES, threadIdx.x, THREADS);
    if (threadIdx.x == 0) stage_tag[s] = panel;
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // Items are numbered row-block-major (item = row block * panels + panel) and dealt out round-robin, CTA c taking
  // items c, c + grid, ...: at any moment the CTAs work on neighbouring panels of the same few row blocks, so whole
  // rows of X are fetched at about the same time (DRAM pages are used in full).  The host sizes the grid so that
  // every ring stage of a CTA keeps meeting the same panel, and with it the transforms it already holds.
  const int item_begin = blockIdx.x, item_step = gridDim.x, item_end = num_items;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    int n = 0;
    for (int it = item_begin; it < item_end; it += item_step, ++n) {
      const int panel = it % num_panels, rb = it / num_panels;
      const int s = n % STAGES;
      const uint32_t ph = (n / STAGES) & 1;
      if (!__all_sync(0xffffffffu, wait(s32(&empty_bar[s]), ph ^ 1, abort_flag))) {
        if (lane == 0) { if (*abort_flag == 0 && status) atomicExch(status, 0x60000 | (n & 0xffff)); *abort_flag = 1; }
        break;
      }
      uint8_t* stage = smem + s * STAGE_BYTES;
      const int nsub = min(SUBS, (int)(K >> 6) - panel * SUBS);        // K tail: the last panel may be one box wide
      const bool dropped = (it == drop_item);                          // test hook, -1 in production
      // the tile first, so that its flight time covers the copy of the transforms below
      if (!dropped && elect()) {
        const uint32_t bar = s32(&full_bar[s]);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(nsub * BOX_BYTES) : "memory");
        for (int sub = 0; sub < nsub; ++sub)
          asm volatile(
              "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
              ::"r"(s32(stage + sub * BOX_BYTES)), "l"(&mapX), "r"((panel * SUBS + sub) * 64), "r"(rb * ROWS), "r"(bar) : "memory");
      }
      __syncwarp();
      if (stage_tag[s] != panel) {                                     // (the first STAGES items were prepared at entry)
        copy_transforms<G, NSPLIT>(T, panel, nsub, stage + X_BYTES, lane, 32);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // written by threads, read by the tensor core
        __syncwarp();
        if (lane == 0) stage_tag[s] = panel;
      }
      __syncwarp();
      // second arrival on the stage's barrier: the transforms it needs are in place
      if (!dropped && lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s32(&full_bar[s])) : "memory");
      __syncwarp();
    }
    if (*abort_flag != 0) {
      // a wait expired somewhere: let every tile that was requested land before the CTA exits
      for (int k = max(0, n - STAGES); k < n; ++k) {
        const uint64_t t0 = timer_ns();
        while (!try_wait(s32(&full_bar[k % STAGES]), (k / STAGES) & 1))
          if (timer_ns() - t0 > 500000000ull) break;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    const uint32_t idesc = idesc_bf16(G);
    int n = 0;
    for (int it = item_begin; it < item_end; it += item_step, ++n) {
      const int panel = it % num_panels;
      const int s = n % STAGES;
      const uint32_t ph = (n / STAGES) & 1;
      // the accumulator buffer has been read out (first round: passes at once), the tile and its transforms are there
      if (!__all_sync(0xffffffffu, wait(s32(&tempty_bar[s]), ph ^ 1, abort_flag)) ||
          !__all_sync(0xffffffffu, wait(s32(&full_bar[s]), ph, abort_flag))) {
        if (lane == 0) { if (*abort_flag == 0 && status) atomicExch(status, 0x70000 | (n & 0xffff)); *abort_flag = 1; }
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (elect()) {
        const int nsub = min(SUBS, (int)(K >> 6) - panel * SUBS);
        for (int sub = 0; sub < nsub; ++sub) {
          const uint64_t adesc = op_desc(s32(smem + s * STAGE_BYTES + sub * BOX_BYTES));
          const uint32_t d = tmem_base + s * ACC_COLS + sub * 64;
#pragma unroll
          for (int b = 0; b < BLOCKS; ++b) {
#pragma unroll
            for (int sp = 0; sp < NSPLIT; ++sp) {            // lo, mid, hi term of the transform (one term for bf16 transforms)
              const uint64_t bdesc = op_desc(s32(smem + s * STAGE_BYTES + X_BYTES + (sub * NSPLIT + sp) * TSUB_BYTES));
#pragma unroll
              for (int ks = 0; ks < G / 16; ++ks) {          // 16 channels (32 bytes) per instruction
                const uint32_t off = (uint32_t)(b * 2 * G + ks * 32) >> 4;
                mma_bf16(d + b * G, adesc + off, bdesc + off, idesc, (sp | ks) != 0);
              }
            }
          }
        }
        commit(s32(&empty_bar[s]));                            // the stage may be refilled once these MMAs are done
        commit(s32(&tfull_bar[s]));                            // ... and the accumulator read
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ epilogue (groups of four warps)
    const int group = (warp - 2) / (4 * SUBS);                 // a group of 4 * SUBS warps per item
    const int sub = ((warp - 2) >> 2) % SUBS;                  // the 64-channel box of the item this warp handles
    const int quarter = warp & 3;                              // tensor-memory lanes 32 * quarter .. + 31
    const int64_t KB = K / G;
    const int ktiles = (int)((KB + 3) >> 2);
    const uint32_t nv_mult_u32 = s32(nv_mult);
    const NvScaleFast nvf = nv_scale_fast(ts);
    float seen = 0.0f;
    int n = 0;
    for (int it = item_begin; it < item_end; it += item_step, ++n) {
      if ((n % (EPI_WARPS / (4 * SUBS))) != group) continue;
      const int cur_panel = it % num_panels, cur_rb = it / num_panels;
      const int s = n % STAGES;
      const uint32_t ph = (n / STAGES) & 1;
      if (!__all_sync(0xffffffffu, wait(s32(&tfull_bar[s]), ph, abort_flag))) {
        if (lane == 0) { if (*abort_flag == 0 && status) atomicExch(status, 0x80000 | (n & 0xffff)); *abort_flag = 1; }
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const bool have = sub < min(SUBS, (int)(K >> 6) - cur_panel * SUBS);     // K tail: this warp's box may not exist
      uint32_t u[2][32];
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + s * ACC_COLS + sub * 64;
      if (have) {
        ld32(taddr, u[0]);
        ld32(taddr + 32, u[1]);
      }
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s32(&tempty_bar[s])) : "memory");

      if (!have) continue;
      const int64_t r = (int64_t)cur_rb * ROWS + quarter * 32 + lane;
      const bool ok = r < M;
      const int box = cur_panel * SUBS + sub;                  // 64-channel box index along K
      if (AMAX) {                                              // AbsMax pass: nothing is quantised or stored
        float a = 0.0f;
#pragma unroll
        for (int i = 0; i < 32; ++i) a = fmaxf(fmaxf(a, fabsf(__uint_as_float(u[0][i]))), fabsf(__uint_as_float(u[1][i])));
        seen = fmaxf(seen, ok ? a : 0.0f);
        continue;
      }
      uint32_t words[8];
      uint32_t sbytes = 0;
#pragma unroll
      for (int b = 0; b < BLOCKS; ++b) {
        const uint32_t byte = quantise_block<G>(&u[(b * G) / 32][(b * G) % 32], mx_ceil, nvf, nv_mult_u32, &words[b * (G / 8)]);
        sbytes |= byte << (8 * b);
      }
      if (!ok) continue;
      // the row's 64 codes = 32 bytes = one full sector, one 256-bit store
      asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                   ::"l"(codes + r * (K >> 1) + (int64_t)box * 32), "r"(words[0]), "r"(words[1]), "r"(words[2]), "r"(words[3]),
                     "r"(words[4]), "r"(words[5]), "r"(words[6]), "r"(words[7]) : "memory");
      const int64_t kb0 = (int64_t)box * BLOCKS;
      uint8_t* sdst = scales + ((sf_layout == 0) ? r * KB + kb0
                                                 : ((r >> 7) * ktiles + (kb0 >> 2)) * 512 + (r & 31) * 16 + ((r & 127) >> 5) * 4 + (kb0 & 3));
      if (G == 32) *reinterpret_cast<uint16_t*>(sdst) = (uint16_t)sbytes;
      else *reinterpret_cast<uint32_t*>(sdst) = sbytes;
    }
    if (AMAX) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) seen = fmaxf(seen, __shfl_xor_sync(0xffffffffu, seen, o));
      if (lane == 0 && ts_out != nullptr) atomicMax(reinterpret_cast<uint32_t*>(ts_out), __float_as_uint(seen));
    }
  }

  // ---- common exit
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace tc

// ------------------------------------------------------------------------------ host side
typedef CUresult (*TcEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                               const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static TcEncodeFn tc_encode_fn() {
  static TcEncodeFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<TcEncodeFn>(p);
  }
  return fn;
}

template <int G, bool AMAX, int NSPLIT>
static cudaError_t tc_launch(const CUtensorMap& map, const void* T, int64_t M, int64_t K, const float* ts, uint8_t* codes,
                             uint8_t* scales, int sf, int num_panels, int n_items, int grid, int32_t* status, int cs, bool pdl,
                             const uint32_t* amax_in, float* ts_out, int mx_ceil, int drop, cudaStream_t st) {
  static bool attr_done_of[kDeviceSlots] = {};           // per instantiation and device
  const int slot = device_slot();
  if (slot < 0) return cudaErrorInvalidDevice;
  constexpr int SMEM = tc::smem_bytes(NSPLIT);
  if (!attr_done_of[slot]) {
    const cudaError_t e = cudaFuncSetAttribute(tc::tq_tc_kernel<G, AMAX, NSPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
    if (e != cudaSuccess) return e;
    attr_done_of[slot] = true;
  }
  if (!pdl) {
    tc::tq_tc_kernel<G, AMAX, NSPLIT><<<grid, tc::THREADS, SMEM, st>>>(map, T, M, K, ts, codes, scales, sf, num_panels, n_items, status, cs,
                                                                        amax_in, ts_out, mx_ceil, drop);
    return cudaGetLastError();
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(tc::THREADS, 1, 1);
  cfg.dynamicSmemBytes = SMEM;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, tc::tq_tc_kernel<G, AMAX, NSPLIT>, map, T, M, K, ts, codes, scales, sf, num_panels, n_items, status, cs,
                            amax_in, ts_out, mx_ceil, drop);
}

// Common host part: tensor map over the bf16 rows, grid size, dispatch.  NSPLIT = 1: T is bf16 (activation side);
// NSPLIT = 3: T is the fp32 weight-side transform.  cudaErrorNotSupported: the caller uses the warp-level kernel.
template <int NSPLIT>
static cudaError_t tc_run(const void* X, int64_t M, int64_t K, const void* T, int g, const float* ts, uint8_t* codes,
                          uint8_t* scales, int sf, int32_t* status, bool clear_status, bool pdl, cudaStream_t st,
                          const QuantOpts& opt) {
  TcEncodeFn enc = tc_encode_fn();
  if (!enc) return cudaErrorNotSupported;
  if ((reinterpret_cast<uintptr_t>(codes) & 31u) != 0) return cudaErrorNotSupported;   // 256-bit code stores
  const int slot = device_slot();
  if (slot < 0) return cudaErrorInvalidDevice;
  static int sm_count_of[kDeviceSlots] = {};
  cudaError_t e;
  if (sm_count_of[slot] == 0) {
    int sms = 0, major = 0;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, slot)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, slot)) != cudaSuccess) return e;
    if (major != 10) return cudaErrorNotSupported;
    sm_count_of[slot] = sms;
  }
  CUtensorMap map;
  const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)tc::ROWS};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(X), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorNotSupported;
  const int num_rb = (int)((M + tc::ROWS - 1) / tc::ROWS);
  const int num_panels = (int)((K / 64 + tc::SUBS - 1) / tc::SUBS);
  const int64_t items = (int64_t)num_panels * num_rb;
  if (items > 0x70000000) return cudaErrorNotSupported;       // item indices are ints and are stepped past the end by up to two grids
  // CTA c takes items c, c + grid, c + 2 grid, ... and item n of a CTA uses ring stage n % STAGES, so a stage sees
  // the panels (c + grid * n) % panels for n = s, s + STAGES, ...: always the same panel when panels divides
  // STAGES * grid, and a stage's transforms are then written once.  The grid is the largest with that property (a
  // multiple of panels / gcd(panels, STAGES): 144 CTAs for K = 8192, 140 for K = 14336), provided it keeps at least
  // 3/4 of the SMs busy.  With the GPU to itself the kernel is bound by HBM and a multiple of the panel count (128,
  // 112 CTAs) is as fast; behind FP4 GEMMs, with the SM clock held down by the power cap, it is bound by the SMs and
  // the larger grid is 9-12 % faster (16384 x 8192: 72.8 -> 66.2 us).
  const int sms = sm_count_of[slot];
  int g4 = tc::STAGES, pp = num_panels;                         // gcd(panels, STAGES)
  while (pp != 0) { const int t = g4 % pp; g4 = pp; pp = t; }
  const int step = num_panels / g4;
  int grid = sms;
  if (step <= sms && (sms / step) * step * 4 >= sms * 3) grid = (sms / step) * step;
  if (items < grid) grid = (int)items;
  const int cs = clear_status ? 1 : 0;
  if (opt.amax_out != nullptr) {                 // AbsMax pass only (g = 16)
    if (g != 16) return cudaErrorNotSupported;
    return tc_launch<16, true, NSPLIT>(map, T, M, K, nullptr, nullptr, nullptr, sf, num_panels, (int)items, grid, status, cs, pdl,
                                       nullptr, reinterpret_cast<float*>(opt.amax_out), 0, -1, st);
  }
  if (g == 32)
    return tc_launch<32, false, NSPLIT>(map, T, M, K, ts, codes, scales, sf, num_panels, (int)items, grid, status, cs, pdl,
                                        opt.amax_in, opt.ts_out, opt.mx_ceil ? 1 : 0, opt.drop_item, st);
  return tc_launch<16, false, NSPLIT>(map, T, M, K, ts, codes, scales, sf, num_panels, (int)items, grid, status, cs, pdl,
                                      opt.amax_in, opt.ts_out, 0, opt.drop_item, st);
}

// Activation side (bf16 transforms).
cudaError_t run_quantize_act_tc(const void* X, int64_t M, int64_t K, const void* T, int g, const float* ts, uint8_t* codes,
                                uint8_t* scales, int sf, int32_t* status, bool clear_status, bool pdl, cudaStream_t st,
                                const QuantOpts& opt) {
  return tc_run<1>(X, M, K, T, g, ts, codes, scales, sf, status, clear_status, pdl, st, opt);
}

// Weight side (Algorithm 2, last line): W[N,K] bf16, Tinv fp32 split three ways inside the kernel.  opt carries the
// AbsMax pass / tensor-scale pointers for NVFP4 exactly as on the activation side.
cudaError_t run_quantize_weight_tc(const void* W, int64_t N, int64_t K, const float* Tinv, int g, uint8_t* codes,
                                   uint8_t* scales, int sf, cudaStream_t st, const QuantOpts& opt) {
  return tc_run<3>(W, N, K, Tinv, g, nullptr, codes, scales, sf, nullptr, false, false, st, opt);
}

}  // namespace wush
