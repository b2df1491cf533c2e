// Streaming variant of the per-block second-moment accumulation (Algorithm 2, RTN case, first line
// of the loop):  S_c += sum_t x_{t,c}^T x_{t,c}  for every block c of g channels.
//
// Same skeleton as the streaming quantiser: persistent CTAs, one producer warp that feeds a 4-stage
// shared-memory ring of 64-token x 128-channel tiles with TMA (two 128-byte-wide boxes, 128-byte
// swizzle, no multicast), 8 consumer warps; two such CTAs share an SM (measured 8 % faster than one
// CTA of 16 consumer warps on 128-token tiles, and than four CTAs of 4).  A work item is
// (128-channel panel, 64-token block); a CTA takes a contiguous run of items in panel-major order.
// Consumer warp (super-block s, token half q) owns the 32 x 32 sum of super-block s over tokens
// 32 q .. 32 q + 31 of every tile it sees.  Tokens are the contraction index of the MMA, so both
// operands are the TRANSPOSE of the stored tile: ldmatrix.trans delivers them in fragment layout
// straight from the row-major tile (A: 16 channels x 16 tokens, B: 16 tokens x two 8-channel tiles),
// no register transposes.  bf16 products are exact in fp32.
//
// When the panel changes (and at the end) the token-part warps of a super-block add their
// sums through shared memory in a fixed order and write one "segment" of partial sums.  Segment k of
// panel p belongs to the k-th CTA (in grid order) that touched panel p; which CTAs those are follows
// from the item count and the grid size alone, so the reduction kernel adds exactly the segments
// that exist, in a fixed order: the result does not depend on scheduling.
//
// Every mbarrier wait is bounded (about one second); a role that gives up raises the CTA's abort
// flag and every role falls through to the exit, where requested copies are allowed to land.
#include <cuda.h>

#include "wush_device.cuh"
#include "wush_host.h"

namespace wush {

constexpr int MS_ROWS = 64;                              // tokens per tile
constexpr int MS_TQ = MS_ROWS / 32;                      // 32-token parts of a tile, one consumer warp each
constexpr int MS_CONSUMERS = 8;
constexpr int MS_CTAS_PER_SM = 16 / MS_CONSUMERS;        // 16 consumer warps per SM either way
constexpr int MS_PANEL_SB = MS_CONSUMERS / MS_TQ;        // 32-channel super-blocks per tile (panel)
constexpr int MS_BOXES = MS_PANEL_SB / 2;                // 64-channel TMA boxes per tile
constexpr int MS_STAGES = 4;
constexpr int MS_THREADS = (MS_CONSUMERS + 1) * 32;
constexpr int MS_BOX_BYTES = MS_ROWS * 128;              // MS_ROWS tokens x 64 channels
constexpr int MS_STAGE_BYTES = MS_BOXES * MS_BOX_BYTES;
constexpr int MS_RED_BYTES = MS_CONSUMERS * 32 * 32 * 4; // one fp32 accumulator set per consumer warp
constexpr int MS_SMEM = MS_STAGES * MS_STAGE_BYTES + MS_RED_BYTES + 1024 + 128;
constexpr int MS_DESIGN_SMS = 148 * MS_CTAS_PER_SM;      // upper bound of the grid (sizes the workspace)

__device__ __forceinline__ uint32_t ms_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ bool ms_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t ms_timer() { uint64_t t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
__device__ __forceinline__ bool ms_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < 2048; ++i)
    if (ms_try_wait(bar, parity)) return true;
  const uint64_t t0 = ms_timer();
  while (true) {
    for (int i = 0; i < 64; ++i)
      if (ms_try_wait(bar, parity)) return true;
    if (*abort_flag != 0 || ms_timer() - t0 > 1000000000ull) return false;
  }
}
__device__ __forceinline__ bool ms_elect() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
  return pred != 0;
}
// four 8x8 matrices of 16-bit elements, transposed on the way: lane l gets (rows 2(l%4), 2(l%4)+1 ; column l/4)
__device__ __forceinline__ uint4 ms_ldmatrix_x4_trans(uint32_t addr) {
  uint4 v;
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// the CTA (of `grid`) whose contiguous run [floor(c I / grid), floor((c+1) I / grid)) holds item `it`
constexpr int MS_FOLD = 32;     // tiles between two folds of the tensor-core sums into the rounded totals
__host__ __device__ __forceinline__ int ms_cta_of_item(int64_t it, int64_t items, int grid) {
  return static_cast<int>(((it + 1) * grid - 1) / items);
}

template <int G>
__global__ void __launch_bounds__(MS_THREADS, MS_CTAS_PER_SM)
moments_stream_kernel(const __grid_constant__ CUtensorMap mapX, int64_t K, float* __restrict__ partials,
                      int num_rb, int num_items) {
  extern __shared__ uint8_t ms_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(ms_raw) + 1023) & ~uintptr_t(1023));
  float* red = reinterpret_cast<float*>(smem + MS_STAGES * MS_STAGE_BYTES);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + MS_STAGES * MS_STAGE_BYTES + MS_RED_BYTES);
  uint64_t* empty_bar = full_bar + MS_STAGES;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(empty_bar + MS_STAGES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 32) prefetch_tensormap(&mapX);
  if (threadIdx.x == 0) {
    for (int s = 0; s < MS_STAGES; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(ms_u32(&full_bar[s])), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(ms_u32(&empty_bar[s])), "r"(MS_CONSUMERS));
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  const int item_begin = (int)(((int64_t)num_items * blockIdx.x) / gridDim.x);
  const int item_end = (int)(((int64_t)num_items * (blockIdx.x + 1)) / gridDim.x);
  const int total_sb = (int)(K >> 5);

  if (warp == MS_CONSUMERS) {
    // ------------------------------------------------------------------ producer warp
    int n = 0;
    int panel = item_begin / num_rb, rb = item_begin % num_rb;
    for (int it = item_begin; it < item_end; ++it, ++n) {
      const int s = n % MS_STAGES;
      const uint32_t ph = (n / MS_STAGES) & 1;
      if (!__all_sync(0xffffffffu, ms_wait(ms_u32(&empty_bar[s]), ph ^ 1, abort_flag))) {
        if (lane == 0) *abort_flag = 1;
        break;
      }
      const int nsb = min(MS_PANEL_SB, total_sb - panel * MS_PANEL_SB);
      if (ms_elect()) {
        const uint32_t bar = ms_u32(&full_bar[s]);
        const int nbox = nsb >> 1;                       // 64-channel (128-byte) boxes; K % 64 == 0
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(nbox * MS_BOX_BYTES) : "memory");
        for (int bx = 0; bx < nbox; ++bx) {
          const uint32_t dst = ms_u32(smem + s * MS_STAGE_BYTES + bx * MS_BOX_BYTES);
          asm volatile(
              "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
              ::"r"(dst), "l"(&mapX), "r"((panel * MS_BOXES + bx) * 64), "r"(rb * MS_ROWS), "r"(bar) : "memory");
        }
      }
      __syncwarp();
      if (++rb == num_rb) { rb = 0; ++panel; }
    }
    if (*abort_flag != 0) {
      // a wait expired somewhere: let every tile that was requested land before the CTA exits
      for (int k = max(0, n - MS_STAGES); k < n; ++k) {
        const uint64_t t0 = ms_timer();
        while (!ms_try_wait(ms_u32(&full_bar[k % MS_STAGES]), (k / MS_STAGES) & 1))
          if (ms_timer() - t0 > 500000000ull) break;
      }
    }
  } else {
    // ------------------------------------------------------------------ consumer warps
    const int gid = lane >> 2, tig = lane & 3;
    const int sbi = warp / MS_TQ;             // super-block of the panel
    const int tq = warp % MS_TQ;              // 32-token part of the tile: tokens 32 tq .. 32 tq + 31
    // ldmatrix.trans operand addresses.  An 8x8 block = 8 token rows x one 16-byte chunk (8 channels) at byte
    // ((chunk ^ (row & 7)) << 4) of its 128-byte box row.  Lane l supplies row (l & 7) of block l >> 3:
    //   A (16 channels x 16 tokens): blocks (tok lo, ch), (tok lo, ch + 8), (tok hi, ch), (tok hi, ch + 8)
    //   B (16 tokens x 2 tiles of 8 channels): blocks (tok lo, ch), (tok hi, ch), (tok lo, ch + 8), (tok hi, ch + 8)
    const uint32_t tile_base = ms_u32(smem) + (sbi >> 1) * MS_BOX_BYTES + (32 * tq) * 128;
    const uint32_t rowA = ((lane & 7) + 8 * (lane >> 4)) * 128, rowB = ((lane & 7) + 8 * ((lane >> 3) & 1)) * 128;
    const uint32_t chA = (lane >> 3) & 1, chB = lane >> 4;
    const uint32_t cbase = 4 * (sbi & 1);     // first chunk of the super-block in its box row
    const uint32_t swz = lane & 7;            // (row & 7) of every row this lane addresses
    constexpr int NT = (G == 32) ? 8 : 4;     // accumulator tiles (16 x 8): g=32: [mt][nt], g=16: [block][nt]
    // Two levels of fp32 sums.  The tensor core adds into `acc` with truncation, a bias of up to one unit in the
    // last place of the running sum per MMA; over the ~10^3 tiles of a CTA's run that reached 1e-4 of a diagonal
    // sum at 2.6e5 tokens.  Every MS_FOLD tiles `acc` is added to `tot` with a rounded fp32 addition and cleared,
    // so the biased sums stay short.
    float acc[NT][4], tot[NT][4];
#pragma unroll
    for (int a = 0; a < NT; ++a) {
      acc[a][0] = acc[a][1] = acc[a][2] = acc[a][3] = 0.f;
      tot[a][0] = tot[a][1] = tot[a][2] = tot[a][3] = 0.f;
    }

    const int64_t seg_stride = K * G;         // floats of one segment of partial sums
    auto flush = [&](int panel) {
      // the four token quarters of a super-block, added in the order 0,1,2,3 by the quarter-0 warp
      float* mine = red + (warp * NT * 4) * 32 + lane;
#pragma unroll
      for (int a = 0; a < NT; ++a)
#pragma unroll
        for (int e = 0; e < 4; ++e) mine[(a * 4 + e) * 32] = __fadd_rn(tot[a][e], acc[a][e]);
      asm volatile("bar.sync 1, %0;" ::"n"(MS_CONSUMERS * 32) : "memory");
      const int sb = panel * MS_PANEL_SB + sbi;
      if (tq == 0 && sb < total_sb) {
        const int seg = (int)blockIdx.x - ms_cta_of_item((int64_t)panel * num_rb, num_items, gridDim.x);
        float* out = partials + (int64_t)seg * seg_stride;
#pragma unroll
        for (int a = 0; a < NT; ++a) {
          float v[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float s = 0.f;
#pragma unroll
            for (int q = 0; q < MS_TQ; ++q) s += red[((warp + q) * NT * 4 + a * 4 + e) * 32 + lane];
            v[e] = (*abort_flag != 0) ? __int_as_float(0x7fc00000) : s;      // a wait expired: make the failure visible (NaN)
          }
          // tile a: g=32: rows 16 (a / 4) + gid (+8), columns 8 (a % 4) + 2 tig (+1) of the 32 x 32 sum;
          //         g=16: block a / 2, rows gid (+8), columns 8 (a % 2) + 2 tig (+1) of its 16 x 16 sum
          if (G == 32) {
            const int i = 16 * (a >> 2) + gid, j = 8 * (a & 3) + 2 * tig;
            *reinterpret_cast<float2*>(out + ((int64_t)sb * 32 + i) * 32 + j) = make_float2(v[0], v[1]);
            *reinterpret_cast<float2*>(out + ((int64_t)sb * 32 + i + 8) * 32 + j) = make_float2(v[2], v[3]);
          } else {
            const int64_t c = (int64_t)sb * 2 + (a >> 1);
            const int j = 8 * (a & 1) + 2 * tig;
            *reinterpret_cast<float2*>(out + (c * 16 + gid) * 16 + j) = make_float2(v[0], v[1]);
            *reinterpret_cast<float2*>(out + (c * 16 + gid + 8) * 16 + j) = make_float2(v[2], v[3]);
          }
        }
      }
      asm volatile("bar.sync 1, %0;" ::"n"(MS_CONSUMERS * 32) : "memory");   // the buffer may be rewritten
#pragma unroll
      for (int a = 0; a < NT; ++a) {
        acc[a][0] = acc[a][1] = acc[a][2] = acc[a][3] = 0.f;
        tot[a][0] = tot[a][1] = tot[a][2] = tot[a][3] = 0.f;
      }
    };

    int n = 0;
    int panel = item_begin / num_rb, rb = item_begin % num_rb;
    int cur_panel = panel;
    bool dead = false;                        // a wait expired: keep walking the items (every consumer warp must
                                              // join the same flush barriers) but touch no tile any more
    for (int it = item_begin; it < item_end; ++it, ++n) {
      if (panel != cur_panel) { flush(cur_panel); cur_panel = panel; }
      const int s = n % MS_STAGES;
      const uint32_t ph = (n / MS_STAGES) & 1;
      if (!dead && !__all_sync(0xffffffffu, ms_wait(ms_u32(&full_bar[s]), ph, abort_flag))) {
        if (lane == 0) *abort_flag = 1;
        dead = true;
      }
      if (dead) {
        if (++rb == num_rb) { rb = 0; ++panel; }
        continue;
      }
      if (panel * MS_PANEL_SB + sbi < total_sb) {       // (K tail: the box of a missing super-block pair is not loaded)
        const uint32_t a0 = tile_base + s * MS_STAGE_BYTES;
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {      // 16 tokens per step
          const uint32_t ra = a0 + ks * (16 * 128) + rowA, rbb = a0 + ks * (16 * 128) + rowB;
          if (G == 32) {
            uint4 A[2], Bf[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {     // channels 16 h .. 16 h + 15 of the super-block
              A[h] = ms_ldmatrix_x4_trans(ra + (((cbase + 2 * h + chA) ^ swz) << 4));
              Bf[h] = ms_ldmatrix_x4_trans(rbb + (((cbase + 2 * h + chB) ^ swz) << 4));
            }
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                mma_bf16_16816(acc[mt * 4 + 2 * h], A[mt].x, A[mt].y, A[mt].z, A[mt].w, Bf[h].x, Bf[h].y);
                mma_bf16_16816(acc[mt * 4 + 2 * h + 1], A[mt].x, A[mt].y, A[mt].z, A[mt].w, Bf[h].z, Bf[h].w);
              }
          } else {
#pragma unroll
            for (int b = 0; b < 2; ++b) {     // the super-block's two 16-channel blocks: only their own products
              const uint4 A = ms_ldmatrix_x4_trans(ra + (((cbase + 2 * b + chA) ^ swz) << 4));
              const uint4 Bf = ms_ldmatrix_x4_trans(rbb + (((cbase + 2 * b + chB) ^ swz) << 4));
              mma_bf16_16816(acc[2 * b], A.x, A.y, A.z, A.w, Bf.x, Bf.y);
              mma_bf16_16816(acc[2 * b + 1], A.x, A.y, A.z, A.w, Bf.z, Bf.w);
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(ms_u32(&empty_bar[s])) : "memory");
      if ((n % MS_FOLD) == MS_FOLD - 1) {
#pragma unroll
        for (int a = 0; a < NT; ++a)
#pragma unroll
          for (int e = 0; e < 4; ++e) { tot[a][e] = __fadd_rn(tot[a][e], acc[a][e]); acc[a][e] = 0.f; }
      }
      if (++rb == num_rb) { rb = 0; ++panel; }
    }
    if (item_end > item_begin) flush(cur_panel);
  }
  __syncthreads();
}

// moments[i] += sum over the segments that exist for element i's panel, in segment order; *count += B
template <int G>
__global__ void moments_reduce_segments_kernel(const float* __restrict__ partials, int64_t n, float* __restrict__ moments,
                                               int64_t* __restrict__ count, int64_t B, int num_rb, int64_t items, int grid) {
  // 256 consecutive elements never straddle a g x g block (256 or 1024 elements), so the whole thread block
  // shares one panel: thread 0 works out how many segments that panel has
  __shared__ int nseg;
  const int64_t i0 = (int64_t)blockIdx.x * blockDim.x;
  if (threadIdx.x == 0) {
    const int64_t c = i0 / (G * G);                                  // block of g channels
    const int64_t panel = (G == 32 ? c : (c >> 1)) / MS_PANEL_SB;    // 32-channel super-blocks per panel
    nseg = ms_cta_of_item((panel + 1) * num_rb - 1, items, grid) - ms_cta_of_item(panel * num_rb, items, grid) + 1;
    if (blockIdx.x == 0 && count != nullptr) *count += B;
  }
  __syncthreads();
  const int64_t i = i0 + threadIdx.x;
  if (i >= n) return;
  float s = 0.f;
  for (int p = 0; p < nseg; ++p) s += partials[(int64_t)p * n + i];
  moments[i] += s;
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*MsEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                               const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static MsEncodeFn ms_encode_fn() {
  static MsEncodeFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<MsEncodeFn>(p);
  }
  return fn;
}

// Segments of partial sums the streaming kernel may write per panel (sizes the workspace): a panel's
// num_rb items are spread over at most ceil(grid / panels) + 1 CTAs, grid <= MS_DESIGN_SMS.
int moments_stream_segments(int64_t B, int64_t K) {
  const int64_t panels = (K / 32 + MS_PANEL_SB - 1) / MS_PANEL_SB;
  const int64_t num_rb = (B + MS_ROWS - 1) / MS_ROWS;
  const int64_t items = panels * num_rb;
  const int64_t grid = items < MS_DESIGN_SMS ? items : MS_DESIGN_SMS;
  int64_t s = (grid + panels - 1) / panels + 1;
  if (s > num_rb) s = num_rb;                 // never more segments than items of a panel
  return (int)(s < 1 ? 1 : s);
}

// Partial sums by the streaming kernel.  *segments_of receives what the reduction needs to know.
// cudaErrorNotSupported: use the register-staged kernel.
cudaError_t run_moments_partial_stream(const void* Xc, int64_t B, int64_t K, int g, float* partials, int slots,
                                       int* grid_out, int* num_rb_out, cudaStream_t st) {
  MsEncodeFn enc = ms_encode_fn();
  if (!enc) return cudaErrorNotSupported;
  const int64_t panels = (K / 32 + MS_PANEL_SB - 1) / MS_PANEL_SB;
  const int64_t num_rb = (B + MS_ROWS - 1) / MS_ROWS;
  const int64_t items = panels * num_rb;
  if (items > 0x7fffffff || B > 0x7fffff00) return cudaErrorNotSupported;
  static int sm_count_of[kDeviceSlots] = {};
  const int slot = device_slot();
  if (slot < 0) return cudaErrorInvalidDevice;
  int& sm_count = sm_count_of[slot];
  cudaError_t e;
  if (sm_count == 0) {
    int dev = slot, sms = 0;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(moments_stream_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, MS_SMEM)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(moments_stream_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, MS_SMEM)) != cudaSuccess) return e;
    sm_count = sms;
  }
  int64_t grid = (int64_t)sm_count * MS_CTAS_PER_SM < MS_DESIGN_SMS ? (int64_t)sm_count * MS_CTAS_PER_SM : MS_DESIGN_SMS;
  // A multiple of the panel count where that keeps at least 3/4 of the slots: every CTA's run is then a stretch of row
  // blocks of ONE panel, the CTAs of neighbouring panels start at the same rows and walk down together, so whole rows
  // of X are fetched at about the same time (DRAM pages used in full) instead of 256-byte pieces of unrelated rows.
  if (panels <= grid && (grid / panels) * panels * 4 >= grid * 3) grid = (grid / panels) * panels;
  if (items < grid) grid = items;
  int64_t need = (grid + panels - 1) / panels + 1;
  if (need > num_rb) need = num_rb;
  if (need > slots) return cudaErrorNotSupported;                       // the caller's workspace holds fewer segments
  CUtensorMap map;
  const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)B};
  const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)MS_ROWS};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(Xc), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorNotSupported;
  if (g == 32)
    moments_stream_kernel<32><<<(unsigned)grid, MS_THREADS, MS_SMEM, st>>>(map, K, partials, (int)num_rb, (int)items);
  else
    moments_stream_kernel<16><<<(unsigned)grid, MS_THREADS, MS_SMEM, st>>>(map, K, partials, (int)num_rb, (int)items);
  *grid_out = (int)grid;
  *num_rb_out = (int)num_rb;
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  return cudaSuccess;
}

// The whole call by the streaming kernels: partial sums, then the segment-aware reduction.
cudaError_t run_calib_moments_stream(const void* Xc, int64_t B, int64_t K, int g, float* moments, int64_t* count,
                                     float* partials, int slots, cudaStream_t st) {
  int grid = 0, num_rb = 0;
  cudaError_t e = run_moments_partial_stream(Xc, B, K, g, partials, slots, &grid, &num_rb, st);
  if (e != cudaSuccess) return e;
  const int64_t panels = (K / 32 + MS_PANEL_SB - 1) / MS_PANEL_SB;
  const int64_t n = K * g;
  const int64_t items = panels * num_rb;
  const unsigned blocks = (unsigned)((n + 255) / 256);
  if (g == 32) moments_reduce_segments_kernel<32><<<blocks, 256, 0, st>>>(partials, n, moments, count, B, num_rb, items, grid);
  else         moments_reduce_segments_kernel<16><<<blocks, 256, 0, st>>>(partials, n, moments, count, B, num_rb, items, grid);
  return cudaGetLastError();
}

}  // namespace wush
