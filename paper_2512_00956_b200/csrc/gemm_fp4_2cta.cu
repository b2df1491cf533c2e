// Block-scaled FP4 GEMM, two-CTA form (Eq. 7, outer sum) - the kernel wush_gemm_fp4 uses for
// M > 128.  Same arithmetic as gemm_fp4.cu; different machine mapping:
//
//  * Persistent clusters of two CTAs (one cluster per SM pair) walk the 256 x 256 output tiles.
//    CTA r of a pair owns rows [128 r, 128 r + 128) of the tile: it loads its 128 rows of A and
//    ITS HALF (128 rows) of the B tile.  tcgen05.mma.cta_group::2 (M = 256, N = 256, K = 64)
//    reads each CTA's B half from that CTA's shared memory, so every SM streams only half of B
//    - a single SM cannot feed its tensor cores at the FP4 rate from its own shared memory -
//    and no TMA multicast is involved anywhere.
//  * All operand and scale loads are TMA tile loads in the cta_group::2 form, which lets both
//    CTAs signal the LEADER's "full" mbarrier.  Two issuing threads work in the leader: one
//    copies each stage's scale tiles to tensor memory (tcgen05.cp.cta_group::2 acts on both
//    CTAs; one 48-column buffer per ring stage), the other issues the MMAs and releases the
//    stage in both CTAs with one multicast tcgen05.commit.
//  * Eight epilogue warps per CTA drain the 128 x 256 fp32 accumulator (tcgen05.ld), signal the
//    leader as soon as the last column has been read, and finish their global stores while the
//    next tile's MMAs already run.  The producers never stop, so the ring is full when they do.
//
// Every mbarrier wait is bounded (about two seconds).  On expiry the role records a diagnostic
// word in *status, raises its CTA's abort flag and falls through to the common exit; the peer
// CTA's own bounded waits expire in turn, so the closing cluster barrier is always reached.
#include <cuda.h>

#include <atomic>

#include "wush_device.cuh"
#include "wush_host.h"

namespace wush {
namespace g2 {

constexpr int BM = 256, BN = 256;       // cluster tile
constexpr int BKB = 128;                // packed-FP4 bytes per row per stage (256 elements)
// Ring depth: as deep as shared memory allows.  A K slab's operands take about 2 us from request to arrival under load
// and 0.27-0.37 us to consume, so the ring is what limits the kernel: MXFP4 stages (35 KB) fit six times, NVFP4 (38 KB) five.
__host__ __device__ constexpr int stages(int fmt) { return fmt == 0 ? 6 : 5; }
constexpr int A_BYTES = 128 * BKB;      // this CTA's 128 rows of A
constexpr int B_BYTES = 128 * BKB;      // this CTA's 128 rows (half) of B
constexpr int EPI_WARPS = 8;
constexpr int SF_WARP = 2 + EPI_WARPS;     // copies scale tiles to tensor memory (leader CTA)
constexpr int THREADS = (3 + EPI_WARPS) * 32;
constexpr uint32_t TMEM_COLS = 512;
// scale tiles: one 48-column buffer per ring stage (A scales 16 columns, B scales 32), after the accumulator
constexpr uint32_t SF_COL0 = 256, SFB_OFF = 16;
// tensor-memory columns of one stage's scale buffer: A 8 / 16 columns from column 0, B 16 / 32 from column 16
__host__ __device__ constexpr uint32_t sf_stride(int fmt) { return fmt == 0 ? 32u : 48u; }
constexpr uint32_t PEER_MASK = 0xFEFFFFFFu;   // clears the CTA-rank bit of a shared::cluster address: rank 0 of the pair

__host__ __device__ constexpr int tps(int fmt) { return fmt == kFmtMX ? 2 : 4; }
__host__ __device__ constexpr int sf_bytes(int fmt) { return 3 * tps(fmt) * 512; }
__host__ __device__ constexpr int stage_bytes(int fmt) { return A_BYTES + B_BYTES + sf_bytes(fmt); }
// rows of one output box: an epilogue warp pushes its 32 rows in two halves where that buys a ring stage (MXFP4)
__host__ __device__ constexpr int epi_rows(int fmt) { return fmt == 0 ? 16 : 32; }
__host__ __device__ constexpr int epi_stage_bytes(int fmt) { return epi_rows(fmt) * 128; }   // per epilogue warp, 128-byte swizzle
// the alignment slack is 768 bytes: the ring must start on a 1 KiB boundary and the dynamic window starts on a 256-byte one
__host__ __device__ constexpr int smem_bytes(int fmt) { return 768 + stages(fmt) * stage_bytes(fmt) + EPI_WARPS * epi_stage_bytes(fmt) + 256; }

__device__ __forceinline__ uint32_t s32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ bool try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t timer_ns() { uint64_t t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
__device__ __forceinline__ bool test_wait(uint32_t bar, uint32_t parity) {   // non-suspending probe: cheaper when the phase is done
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < 16; ++i)
    if (test_wait(bar, parity)) return true;
  for (int i = 0; i < 4096; ++i)
    if (try_wait(bar, parity)) return true;
  const uint64_t t0 = timer_ns();
  while (true) {
    for (int i = 0; i < 64; ++i)
      if (try_wait(bar, parity)) return true;
    if (*abort_flag != 0 || timer_ns() - t0 > 2000000000ull) return false;
  }
}
__device__ __forceinline__ bool elect() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
  return pred != 0;
}
// TMA tile load whose completion bytes are counted on the pair leader's mbarrier (no multicast)
__device__ __forceinline__ void tma_2sm(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t leader_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(leader_bar) : "memory");
}
__device__ __forceinline__ void commit_both(uint32_t bar) {      // arrives on `bar` in both CTAs of the pair
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void commit_leader(uint32_t bar) {    // arrives on the leader's `bar` only
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)1) : "memory");
}
__device__ __forceinline__ void arrive_leader(uint32_t bar) {    // one arrival on the leader's copy of `bar`
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar & PEER_MASK) : "memory");
}
__device__ __forceinline__ void cp_sf2(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
template <int FMT>
__device__ __forceinline__ void mma2(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t sfa, uint32_t sfb, uint32_t acc) {
  if (FMT == kFmtMX) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc), "r"(sfa), "r"(sfb) : "memory");
  } else {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.scale_vec::4X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc), "r"(sfa), "r"(sfb) : "memory");
  }
}
__device__ __forceinline__ void ld32(uint32_t taddr, uint32_t (&r)[32]) {
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
__device__ __forceinline__ uint64_t op_desc(uint32_t a) {      // K-major, 128-byte swizzle, 8-row groups 1024 B apart
  return static_cast<uint64_t>((a & 0x3FFFFu) >> 4) | (1ull << 16) | (static_cast<uint64_t>(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint64_t sf_desc(uint32_t a) {      // 32 rows x 16 B, no swizzle
  return static_cast<uint64_t>((a & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(128 >> 4) << 32) | (1ull << 46);
}
__device__ __forceinline__ uint32_t idesc2(int fmt, uint32_t sf_byte) {   // M = 256 across the pair, N = 256
  return (sf_byte << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
         ((fmt == kFmtMX ? 1u : 0u) << 23) | (static_cast<uint32_t>(BM >> 4) << 24) | (sf_byte << 29);
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}

// Tile order.  The clusters work on consecutive tile indices at any one time, so the order decides what the L2
// holds: row-major order makes ~74 concurrent tiles share one 256-row panel of A and touch 74 different panels
// of B, i.e. the whole of B streams from HBM once per row of tiles.  Here the tiles are walked in bands of
// RASTER_M tile rows, column by column inside a band: the concurrent tiles then cover RASTER_M panels of A and
// about 74 / RASTER_M panels of B, and B is read from HBM once per BAND.
constexpr int RASTER_M = 8;
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int& tm, int& tn) {
  const int per_band = RASTER_M * tiles_n;
  const int band = tile / per_band, in_band = tile - band * per_band;
  const int first = band * RASTER_M;
  const int rows = min(RASTER_M, tiles_m - first);      // the last band may be shorter
  tn = in_band / rows;
  tm = first + (in_band - tn * rows);
}

template <int FMT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
gemm_fp4_2cta_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                     const __grid_constant__ CUtensorMap mapSFA, const __grid_constant__ CUtensorMap mapSFB,
                     int M, int N, int K, const float* __restrict__ tsx, const float* __restrict__ tsw,
                     const __grid_constant__ CUtensorMap mapY, int out_bf16, int32_t* __restrict__ status, int clear_status) {
  constexpr int TPS = tps(FMT);
  constexpr int STAGES = stages(FMT);
  constexpr uint32_t SF_STRIDE = sf_stride(FMT);
  constexpr int EPI_ROWS = epi_rows(FMT), EPI_STAGE_BYTES = epi_stage_bytes(FMT);
  constexpr int KSTEPS_PER_TILE = (FMT == kFmtMX) ? 2 : 1;
  extern __shared__ uint8_t raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = sA + STAGES * A_BYTES;
  uint8_t* sSF = sB + STAGES * B_BYTES;
  uint8_t* sEpi = sSF + STAGES * sf_bytes(FMT);     // 1024-byte aligned: all sizes above are multiples of 1 KiB
  uint64_t* bars = reinterpret_cast<uint64_t*>(sEpi + EPI_WARPS * EPI_STAGE_BYTES);
  uint64_t* full_bar = bars;                      // used in the leader only
  uint64_t* empty_bar = bars + STAGES;            // one copy per CTA, released together by the multicast commit
  uint64_t* tmem_full = bars + 2 * STAGES;        // per CTA
  uint64_t* tmem_empty = bars + 2 * STAGES + 1;   // leader only: 2 x EPI_WARPS arrivals per tile
  uint64_t* sf_full = bars + 2 * STAGES + 2;      // leader only: scale tiles of a stage are in tensor memory
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 3 * STAGES + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  {
    // The window is sized with 768 bytes to spare for the 1 KiB alignment of the ring.  Its start is the same in
    // every CTA of the grid, so if it ever sat less than 256-byte aligned all CTAs leave here together, before any
    // barrier or tensor memory exists, and the call reports it.
    uint32_t dyn;
    asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    if (static_cast<uint32_t>(smem - raw) + smem_bytes(FMT) - 768 > dyn) {
      if (threadIdx.x == 0 && blockIdx.x == 0 && status) atomicExch(status, 0x160000);
      return;
    }
  }
  const uint32_t rank = cluster_rank();            // 0 = leader
  const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
  const int tiles_n = (N + BN - 1) / BN, tiles_m = (M + BM - 1) / BM;
  const int num_tiles = tiles_m * tiles_n;
  const int num_kb = (K + 2 * BKB - 1) / (2 * BKB);
  const int sf_cols = K / (FMT == kFmtMX ? 32 : 16);
  const int ktiles_total = (sf_cols + 3) >> 2;

  if (threadIdx.x == 32 * SF_WARP) {             // descriptors on their way while the barriers and TMEM are set up
    prefetch_tensormap(&mapB); prefetch_tensormap(&mapSFB); prefetch_tensormap(&mapA); prefetch_tensormap(&mapSFA);
    prefetch_tensormap(&mapY);
    // stand-alone call: clear the status word here (a report can only follow a wait of about two seconds, so
    // this cannot erase one); inside wush_linear the quantiser kernel has cleared it
    if (clear_status && blockIdx.x == 0 && status != nullptr) *status = 0;
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(&full_bar[s])), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(&empty_bar[s])), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(&sf_full[s])), "r"(1));
    }
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(tmem_full)), "r"(1));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(tmem_empty)), "r"(2 * EPI_WARPS));
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync();                                  // both CTAs' barriers exist before anything remote touches them
  // a programmatic dependent (the next layer's quantiser) may be scheduled as SMs free up; it waits for this
  // whole grid before it touches memory
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer (one per CTA)
    int g = 0;                                     // running k-block count across tiles
    bool ok = true;
    // weight side of a stage (the leader also announces the stage's whole byte count), activation side
    auto weights = [&](int kb, int s, int n0) {
      const uint32_t bar = s32(&full_bar[s]) & PEER_MASK;            // the leader's barrier
      if (rank == 0)
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(&full_bar[s])), "r"(2 * stage_bytes(FMT)) : "memory");
      uint8_t* sf = sSF + s * sf_bytes(FMT);
      tma_2sm(s32(sB + s * B_BYTES), &mapB, kb * BKB, n0 + (int)rank * 128, bar);
      tma_2sm(s32(sf + TPS * 512), &mapSFB, 0, (n0 >> 7) * ktiles_total + kb * TPS, bar);
      tma_2sm(s32(sf + 2 * TPS * 512), &mapSFB, 0, ((n0 >> 7) + 1) * ktiles_total + kb * TPS, bar);
    };
    auto activations = [&](int kb, int s, int m0) {
      const uint32_t bar = s32(&full_bar[s]) & PEER_MASK;
      uint8_t* sf = sSF + s * sf_bytes(FMT);
      tma_2sm(s32(sA + s * A_BYTES), &mapA, kb * BKB, m0, bar);
      tma_2sm(s32(sf), &mapSFA, 0, (m0 >> 7) * ktiles_total + kb * TPS, bar);
    };
    // Launched as a programmatic dependent of the quantiser (wush_linear), everything above overlapped with
    // that kernel's tail.  The weights do not depend on it: the first ring-full of weight tiles is requested
    // before the wait, the quantiser's output only after it.  The wait is a no-op for a plain launch.
    const int pre = (cluster_id < num_tiles) ? min(STAGES, num_kb) : 0;
    if (pre > 0) {
      int tm, tn;
      tile_coords(cluster_id, tiles_m, tiles_n, tm, tn);
      const int m0 = tm * BM + (int)rank * 128;
      const int n0 = tn * BN;
      if (elect())
        for (int kb = 0; kb < pre; ++kb) weights(kb, kb, n0);
      __syncwarp();
      asm volatile("griddepcontrol.wait;" ::: "memory");
      if (elect())
        for (int kb = 0; kb < pre; ++kb) activations(kb, kb, m0);
      __syncwarp();
    }
    for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
      int tm, tn;
      tile_coords(tile, tiles_m, tiles_n, tm, tn);
      const int m0 = tm * BM + (int)rank * 128;
      const int n0 = tn * BN;
      for (int kb = (tile == cluster_id ? pre : 0); kb < num_kb; ++kb) {
        g = ((tile - cluster_id) / num_clusters) * num_kb + kb;
        const int s = g % STAGES;
        const uint32_t ph = (g / STAGES) & 1;
        if (!__all_sync(0xffffffffu, wait(s32(&empty_bar[s]), ph ^ 1, abort_flag))) {
          if (lane == 0) { if (*abort_flag == 0 && status) atomicExch(status, 0x110000 | (rank << 15) | (g & 0x7fff)); *abort_flag = 1; }
          ok = false;
          break;
        }
        if (elect()) {
          weights(kb, s, n0);
          activations(kb, s, m0);
        }
        __syncwarp();
      }
    }
    if (!ok && rank == 0) {
      // A wait expired.  Copies this pair has already requested must land before either CTA exits: all of them
      // (both CTAs') count on the leader's full barriers, so the leader waits for the stages requested so far,
      // with one deadline for all of them, and the peer stays at the closing cluster barrier until the leader
      // arrives there.  A stage the peer never requested simply runs into the deadline.
      const uint64_t t0 = timer_ns();
      for (int k = max(0, g - STAGES); k < g; ++k)
        while (!try_wait(s32(&full_bar[k % STAGES]), (k / STAGES) & 1))
          if (timer_ns() - t0 > 2000000ull) break;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (rank == 0) {
      int g = 0, it = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++it) {
        if (it > 0) {                               // the epilogues of both CTAs have drained the accumulator
          if (!__all_sync(0xffffffffu, wait(s32(tmem_empty), (it - 1) & 1, abort_flag))) {
            if (lane == 0) { if (*abort_flag == 0 && status) atomicExch(status, 0x130000 | (it & 0xffff)); *abort_flag = 1; }
            ok = false;
            break;
          }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        }
        for (int kb = 0; kb < num_kb; ++kb, ++g) {
          const int s = g % STAGES;
          const uint32_t ph = (g / STAGES) & 1;
          // the scale warp has seen this stage's operands land and has copied its scale tiles to tensor memory
          if (!__all_sync(0xffffffffu, wait(s32(&sf_full[s]), ph, abort_flag))) {
            if (lane == 0) { if (*abort_flag == 0 && status) atomicExch(status, 0x120000 | (g & 0xffff)); *abort_flag = 1; }
            ok = false;
            break;
          }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const int ksteps = min(4, (K - kb * 2 * BKB) / 64);
          const uint64_t adesc = op_desc(s32(sA + s * A_BYTES));
          const uint64_t bdesc = op_desc(s32(sB + s * B_BYTES));
          const uint32_t sfa_t = tmem_base + SF_COL0 + SF_STRIDE * s, sfb_t = sfa_t + SFB_OFF;
          if (elect()) {
            for (int j = 0; j < ksteps; ++j) {
              const int t4 = j / KSTEPS_PER_TILE;
              const uint32_t sfb = (FMT == kFmtMX) ? 2u * (j % KSTEPS_PER_TILE) : 0u;
              mma2<FMT>(tmem_base, adesc + 2 * j, bdesc + 2 * j, idesc2(FMT, sfb), sfa_t + 4 * t4, sfb_t + 8 * t4, (kb | j) != 0);
            }
            commit_both(s32(&empty_bar[s]));
          }
          __syncwarp();
        }
        if (!ok) break;
        if (elect()) commit_both(s32(tmem_full));
        __syncwarp();
      }
    }
  } else if (warp == SF_WARP) {
    // ------------------------------------------------------------------ scale-tile copier (leader CTA only)
    // A second issuing thread: tcgen05.cp costs about as many issue cycles per K slab as the MMAs do, so the
    // copies run from their own warp.  Buffer s of tensor memory belongs to ring stage s: when stage s has
    // been refilled, the MMAs that read its previous scales have completed (that is what freed the stage).
    if (rank == 0) {
      int g = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
        for (int kb = 0; kb < num_kb; ++kb, ++g) {
          const int s = g % STAGES;
          const uint32_t ph = (g / STAGES) & 1;
          if (!__all_sync(0xffffffffu, wait(s32(&full_bar[s]), ph, abort_flag))) {
            if (lane == 0) { if (*abort_flag == 0 && status) atomicExch(status, 0x150000 | (g & 0xffff)); *abort_flag = 1; }
            ok = false;
            break;
          }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const int tiles = min(TPS, ktiles_total - kb * TPS);
          const uint32_t sf = s32(sSF + s * sf_bytes(FMT));
          const uint32_t sfa_t = tmem_base + SF_COL0 + SF_STRIDE * s, sfb_t = sfa_t + SFB_OFF;
          if (elect()) {
            for (int i = 0; i < tiles; ++i) {
              cp_sf2(sfa_t + 4 * i, sf_desc(sf + i * 512));
              cp_sf2(sfb_t + 8 * i, sf_desc(sf + (TPS + i) * 512));
              cp_sf2(sfb_t + 8 * i + 4, sf_desc(sf + (2 * TPS + i) * 512));
            }
            commit_leader(s32(&sf_full[s]));
          }
          __syncwarp();
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (8 warps per CTA)
    const int q = warp & 3;                        // tensor-memory lane quarter this warp may read
    const int half = (warp - 2) >> 2;              // columns [128 half, 128 half + 128)  (warps 2..9)
    // the activation tensor scale may have been written by the preceding kernel of the stream (per-batch
    // scale): as a programmatic dependent this grid may read it only after that kernel has completed
    asm volatile("griddepcontrol.wait;" ::: "memory");
    float alpha = 1.0f;
    if (FMT == kFmtNV) alpha = __fmul_rn(*tsx, *tsw);
    int it = 0;
    bool ok = true;
    for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++it) {
      int tm, tn;
      tile_coords(tile, tiles_m, tiles_n, tm, tn);
      const int m0 = tm * BM + (int)rank * 128;
      const int n0 = tn * BN + half * 128;
      if (!__all_sync(0xffffffffu, wait(s32(tmem_full), it & 1, abort_flag))) {
        if (lane == 0) { if (*abort_flag == 0 && status) atomicExch(status, 0x140000 | (rank << 15) | (it & 0x7fff)); *abort_flag = 1; }
        ok = false;
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // Read this warp's whole 32-lane x 128-column slice into registers first and hand the accumulator
      // back at once: the row-scattered global stores below are slow (one sector per lane and
      // instruction) and must not hold up the next tile's MMAs.
      uint32_t r[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c)
        ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + half * 128 + c * 32, r[c]);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) arrive_leader(s32(tmem_empty));
      // Store through shared memory and TMA: the warp (for MXFP4 half of it at a time, the buffer being kept at 16
      // rows so that the operand ring can have one more stage) writes its rows x 128 bytes (swizzled, so the 16-byte
      // row pieces spread over all banks) and one lane hands the box to the TMA unit, which writes whole 128-byte
      // lines and clips rows >= M and columns >= N by itself.
      uint8_t* stage = sEpi + (warp - 2) * EPI_STAGE_BYTES;
      const uint32_t stage_u32 = s32(stage);
      auto push_box = [&](int col, int row) {             // buffer filled: hand it to the TMA unit
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                       ::"l"(&mapY), "r"(col), "r"(row), "r"(stage_u32) : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      };
      auto buffer_free = [&]() {                          // the previous box has been read out of the buffer
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
      };
      uint8_t* my_row = stage + (lane & (EPI_ROWS - 1)) * 128;
      const int my_half = lane / EPI_ROWS;
      if (out_bf16) {
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {                 // 64 columns (128 bytes of bf16) per box
          const int col = n0 + sub * 64;
          if (col >= N) continue;                           // warp-uniform
#pragma unroll
          for (int h = 0; h < 32 / EPI_ROWS; ++h) {
            const int row = m0 + q * 32 + h * EPI_ROWS;
            if (row >= M) break;                            // warp-uniform
            buffer_free();
            if (my_half == h) {
#pragma unroll
              for (int j = 0; j < 8; ++j) {                 // chunk j = columns 8j..8j+7 = r[2*sub + j/4][8*(j%4)..]
                uint32_t p[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(r[2 * sub + (j >> 2)][8 * (j & 3) + 2 * e]) * alpha,
                                                           __uint_as_float(r[2 * sub + (j >> 2)][8 * (j & 3) + 2 * e + 1]) * alpha);
                  p[e] = *reinterpret_cast<uint32_t*>(&v);
                }
                *reinterpret_cast<uint4*>(my_row + ((j ^ (lane & 7)) << 4)) = make_uint4(p[0], p[1], p[2], p[3]);
              }
            }
            push_box(col, row);
          }
        }
      } else {
#pragma unroll
        for (int sub = 0; sub < 4; ++sub) {                 // 32 columns (128 bytes of fp32) per box
          const int col = n0 + sub * 32;
          if (col >= N) continue;                           // warp-uniform
#pragma unroll
          for (int h = 0; h < 32 / EPI_ROWS; ++h) {
            const int row = m0 + q * 32 + h * EPI_ROWS;
            if (row >= M) break;                            // warp-uniform
            buffer_free();
            if (my_half == h) {
#pragma unroll
              for (int j = 0; j < 8; ++j)
                *reinterpret_cast<uint4*>(my_row + ((j ^ (lane & 7)) << 4)) =
                    make_uint4(__float_as_uint(__uint_as_float(r[sub][4 * j]) * alpha), __float_as_uint(__uint_as_float(r[sub][4 * j + 1]) * alpha),
                               __float_as_uint(__uint_as_float(r[sub][4 * j + 2]) * alpha), __float_as_uint(__uint_as_float(r[sub][4 * j + 3]) * alpha));
            }
            push_box(col, row);
          }
        }
      }
    }
    // every box has been read out of shared memory before the CTA may exit; the writes themselves complete
    // with the grid
    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  }

  // ---- common exit: nobody leaves while the peer may still touch this CTA's memory or barriers
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace g2

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                          const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                          CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncFn enc_fn() {
  static EncFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncFn>(p);
  }
  return fn;
}
static bool map_bytes(CUtensorMap* map, const void* base, int64_t rows, int64_t row_bytes, int box_rows) {
  const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
  const cuuint32_t box[2] = {(cuuint32_t)g2::BKB, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return enc_fn()(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// scale buffer as [tiles][128 x int32]: one row per 512-byte scale tile, box = `tiles_per_box` tiles
static bool map_scales(CUtensorMap* map, const void* base, int64_t total_tiles, int tiles_per_box) {
  const cuuint64_t dims[2] = {128, (cuuint64_t)total_tiles};
  const cuuint64_t strides[1] = {512};
  const cuuint32_t box[2] = {128, (cuuint32_t)tiles_per_box};
  const cuuint32_t estr[2] = {1, 1};
  return enc_fn()(map, CU_TENSOR_MAP_DATA_TYPE_INT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// output [M][N] bf16 or fp32; box = 128 bytes x 16 (MXFP4) or 32 (NVFP4) rows, 128-byte swizzle
static bool map_output(CUtensorMap* map, void* Y, int64_t M, int64_t N, int out_bf16, int fmt) {
  const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)N * (out_bf16 ? 2 : 4)};
  const cuuint32_t box[2] = {(cuuint32_t)(out_bf16 ? 64 : 32), (cuuint32_t)g2::epi_rows(fmt)};
  const cuuint32_t estr[2] = {1, 1};
  return enc_fn()(map, out_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, Y, dims, strides,
                  box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static std::atomic<int> g_cluster_limit[kDeviceSlots];
int gemm_2cta_cluster_limit(int clusters) {
  const int slot = device_slot();
  if (slot < 0) return 0;
  return g_cluster_limit[slot].exchange(clusters < 0 ? 0 : clusters);
}

template <int FMT>
static cudaError_t launch_2cta(const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& sa, const CUtensorMap& sb,
                               int M, int N, int K, const float* tsx, const float* tsw, const CUtensorMap& y, int out_bf16,
                               int32_t* status, bool clear_status, bool pdl, cudaStream_t st) {
  static int clusters_of[kDeviceSlots] = {};       // resident clusters of this kernel, per device
  const int slot = device_slot();
  if (slot < 0) return cudaErrorInvalidDevice;
  int& clusters = clusters_of[slot];
  const int cs = clear_status ? 1 : 0;
  cudaError_t e;
  if (clusters == 0) {
    e = cudaFuncSetAttribute(g2::gemm_fp4_2cta_kernel<FMT>, cudaFuncAttributeMaxDynamicSharedMemorySize, g2::smem_bytes(FMT));
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sms & ~1, 1, 1);
    cfg.blockDim = dim3(g2::THREADS, 1, 1);
    cfg.dynamicSmemBytes = g2::smem_bytes(FMT);
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, g2::gemm_fp4_2cta_kernel<FMT>, &cfg);
    if (e != cudaSuccess || n <= 0) { (void)cudaGetLastError(); n = sms / 2; }
    clusters = n < sms / 2 ? n : sms / 2;
  }
  const int tiles = ((M + g2::BM - 1) / g2::BM) * ((N + g2::BN - 1) / g2::BN);
  int nc = tiles < clusters ? tiles : clusters;
  const int limit = g_cluster_limit[slot].load();
  if (limit > 0 && limit < nc) nc = limit;
  if (!pdl) {
    g2::gemm_fp4_2cta_kernel<FMT><<<2 * nc, g2::THREADS, g2::smem_bytes(FMT), st>>>(a, b, sa, sb, M, N, K, tsx, tsw, y,
                                                                                     out_bf16, status, cs);
    return cudaGetLastError();
  }
  // programmatic dependent launch: this grid may start while the preceding kernel of the stream drains
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * nc, 1, 1);
  cfg.blockDim = dim3(g2::THREADS, 1, 1);
  cfg.dynamicSmemBytes = g2::smem_bytes(FMT);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, g2::gemm_fp4_2cta_kernel<FMT>, a, b, sa, sb, M, N, K, tsx, tsw, y, out_bf16, status, cs);
}

// cudaErrorNotSupported: the caller should use the single-CTA kernel.
cudaError_t run_gemm_fp4_2cta(const uint8_t* Xq, const uint8_t* Xs, const uint8_t* Wq, const uint8_t* Ws, int64_t M,
                              int64_t N, int64_t K, int fmt, const float* tsx, const float* tsw, void* Y,
                              int out_bf16, int32_t* status, bool clear_status, bool pdl, cudaStream_t st) {
  if (!enc_fn()) return cudaErrorNotSupported;
  const int64_t ktiles = ((K / (fmt == kFmtMX ? 32 : 16)) + 3) / 4;
  CUtensorMap a, b, sa, sb, y;
  if (!map_output(&y, Y, M, N, out_bf16, fmt) || !map_bytes(&a, Xq, M, K / 2, 128) || !map_bytes(&b, Wq, N, K / 2, 128) ||
      !map_scales(&sa, Xs, ((M + 127) / 128) * ktiles, g2::tps(fmt)) ||
      !map_scales(&sb, Ws, ((N + 127) / 128) * ktiles, g2::tps(fmt)))
    return cudaErrorNotSupported;
  if (fmt == kFmtMX) return launch_2cta<kFmtMX>(a, b, sa, sb, (int)M, (int)N, (int)K, tsx, tsw, y, out_bf16, status, clear_status, pdl, st);
  return launch_2cta<kFmtNV>(a, b, sa, sb, (int)M, (int)N, (int)K, tsx, tsw, y, out_bf16, status, clear_status, pdl, st);
}

}  // namespace wush
