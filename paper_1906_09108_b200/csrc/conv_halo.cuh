// 3x3 / stride 1 / pad 1 convolutions of narrow layers (16, 32 or 64 channels per pixel) on the
// sm_100a tensor cores, organised around a HALO TILE: one TMA load brings G whole images, each
// with its one-pixel zero border (the hardware's out-of-bounds fill is the padding), into shared
// memory as consecutive "padded pixels" of one swizzle span each (32/64/128 bytes).  Every filter
// tap is then the same tile seen from a start address shifted by (r*Wp + s) pixels, so an
// activation is read from L2/HBM once per pass instead of once per tap.
//
//   padded pixel index  q = (g*Hp + h')*Wp + w'      Hp = H+2, Wp = W+2
//   output pixel (g,h,w) has accumulator row  m = (g*Hp + h)*Wp + w  and reads q = m + r*Wp + s
//   rows m with w >= W or h >= H are computed but never stored.
//
// Forward / data gradient (conv_halo_kernel):
//   D[m][n] = sum_tap sum_c X[m + r*Wp + s][c] * Wt[tap][n][c]       (both operands K-major)
//   M = 128 padded pixels per accumulator, N = output channels, K = 16 channels per instruction.
//   The data gradient is the same kernel on dy with the flipped/transposed weight copy.
// Weight gradient (wgrad_halo_kernel):
//   dW[n][r][s][c] = sum_q dY[q][n] * X[q + r*Wp + s][c]
//   pixels are the reduction dimension, so both operands are read MN-major from the same kind of
//   tile; the A operand stacks the filter taps of one filter row along M (its M-blocks start one
//   pixel apart), B is dY with its border columns and rows zero.  Each CTA keeps its partial sums
//   in tensor memory over all its tiles, writes them once, and a fixed-order pass adds the CTAs'
//   partials, so the result does not depend on scheduling.
//
// Roles by warp: 0 = TMA producer, 1..2 = MMA issuers (one elected lane each, alternate 128-row
// tiles), 3..14 = epilogue (three groups of four warps, 32 tensor-memory lanes per warp).  Every
// wait is bounded; on time-out the CTA raises an error word.
#pragma once
#include "conv_tc.cuh"
#include "elementwise.cuh"

namespace fdg {
namespace halo {

using namespace fdg::tc;

struct FwdParams {
  int W, H, N, Wp, Hp;
  int Ck, Cn;                 // channels of the activation operand (16/32/64) and of the output
  int G;                      // images per tile
  int tiles;                  // ceil(N / G)
  int m_tiles;                // 128-row accumulators per tile
  int img_rows;               // Hp * Wp
  uint32_t pitch;             // Ck * 2 bytes = swizzle span
  uint32_t tile_tx_bytes;     // bytes one TMA tile load writes
  uint32_t stage_bytes;       // shared memory reserved per stage (multiple of 1024)
  int stages;
  uint32_t w_tap_bytes;       // shared memory reserved per filter tap of the weights (multiple of 1024)
  uint32_t w_tx_bytes;        // bytes one weight-tap load writes
  int nacc;                   // accumulator slots in tensor memory
  uint32_t tmem_cols;
  int sub;                    // 1, or 2: keep only the pixels with even h and w and store them as an
                              // [N][H/2][W/2][Cn] tensor (a stride-2 convolution is the stride-1 one subsampled)
};

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Asks for `bytes` (a multiple of 16, from a 16-byte aligned address) to be brought into L2.
__device__ __forceinline__ void prefetch_l2_bulk(const void* p, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

// Shared-memory descriptor of an MN-major operand made of swizzle-span-wide rows (one per k):
// `lbo` = byte distance between consecutive MN blocks, 8-row k groups `8*row_bytes` apart.
__device__ __forceinline__ uint64_t smem_desc_mnmajor(uint32_t addr, uint32_t row_bytes, uint32_t lbo) {
  const uint64_t layout = row_bytes == 128 ? 2 : (row_bytes == 64 ? 4 : 6);
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)(((8 * row_bytes) >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= layout << 61;
  return d;
}
// bf16 x bf16 -> fp32, M = 128; `mn_major` sets both operands MN-major.
__device__ __forceinline__ uint32_t instr_desc(int n, bool mn_major) {
  uint32_t d = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
  if (mn_major) d |= (1u << 15) | (1u << 16);
  return d;
}

// Optional per-channel reduction over the tensor the kernel stores, taken in its epilogue (on
// the values as stored, i.e. after rounding to bf16):
//   mode 1  batch-norm statistics of the output:  sum v, sum v^2
//   mode 2  the two sums of the batch-norm backward the output feeds as its upstream gradient:
//           dz = v * [mask > 0],  sum dz,  sum dz * xhat  with xhat = (xprev - mean) * invstd
// Every CTA writes its sums to partial[cta][2*Cn]; the kernel that consumes the totals adds the
// CTAs' rows in CTA order (elementwise.cuh, finalize_partials), so the result does not depend on
// scheduling and no grid-wide synchronisation is needed here.  Cn <= 64 only.
struct EpiReduce {
  int mode;
  const __nv_bfloat16* mask;
  const __nv_bfloat16* xprev;
  const float* pstats;        // mode 2: mean[Cn], invstd[Cn] of xprev's batch norm
  float* partial;             // [gridDim.x][2*Cn]
};
// Threads of conv_halo_kernel: TMA warp, two MMA warps, kEpiGroups groups of four epilogue warps.
// The groups take the (128-row tile, 16-column chunk) items in turn: an item's epilogue is a chain
// of dependent steps (wait, tensor-memory load, shuffles), so several must be in flight.  Three
// groups divide the 9 tiles of a 32x32 image evenly and leave each thread the registers to hold
// the next item's global operands while it works on the current one.
constexpr int kEpiGroups = 3;
constexpr int kEpiWarps = 4 * kEpiGroups;
// One thread can issue a tcgen05.mma every ~75 cycles, the tensor pipe takes one of these small
// instructions every ~40: two issuing warps (alternate 128-row tiles) keep it busier (measured).
constexpr int kMmaWarps = 2;
constexpr int kFirstEpiWarp = 1 + kMmaWarps;
constexpr int kFwdThreads = 32 * (kFirstEpiWarp + kEpiWarps);
constexpr int kRedSmemBytes = kEpiWarps * 8 * 32 * 4 + 2 * 128 * 4;   // running sums, statistics
// conv_halo_kernel: four issuing warps, one per warp scheduler (a warp's scheduler and its tensor-memory lane
// quarter are both warp % 4, so every scheduler also hosts epilogue warps, and an issuing thread competes with
// them for issue slots: while the epilogue of earlier tiles runs, one issuer gets an instruction out only every
// ~150 cycles; four of them keep the pipe fed).  Warp 0's issuing thread is also the TMA producer.
constexpr int kConvMmaWarps = 4;
constexpr int kConvFirstEpiWarp = kConvMmaWarps;
constexpr int kConvThreads = 32 * (kConvFirstEpiWarp + kEpiWarps);

// The 9 * KS instructions of one 128-row tile, fully unrolled (the issuing thread is the
// bottleneck: every instruction it spends per tcgen05.mma beyond the add and the issue shows).
template <int KS>
__device__ __forceinline__ void issue_tile(uint32_t d_tmem, uint64_t x_desc, const uint64_t (&tap_off)[9], uint64_t w_desc0,
                                           uint64_t w_tap_step, uint32_t idesc) {
#pragma unroll
  for (int tap = 0; tap < 9; ++tap) {
    const uint64_t a0 = x_desc + tap_off[tap], b0 = w_desc0 + tap * w_tap_step;
#pragma unroll
    for (int j = 0; j < KS; ++j) tc_mma_bf16(d_tmem, a0 + 2 * j, b0 + 2 * j, idesc, (tap | j) != 0);
  }
}

// ------------------------------------------------------- forward / data gradient --
// out[pixel][n] (bf16, row stride Cn) = conv + (res ? res * [mask ? mask > 0 : 1] : 0)
__global__ void __launch_bounds__(kConvThreads, 1)
conv_halo_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, FwdParams p,
                 __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ res,
                 const __nv_bfloat16* __restrict__ res_mask, EpiReduce red, int* __restrict__ error_word) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* w_smem = smem + (size_t)p.stages * p.stage_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(w_smem + 9 * (size_t)p.w_tap_bytes);
  uint64_t* full = bars;                       // [stages]  TMA -> MMA
  uint64_t* empty = full + p.stages;           // [stages]  MMA -> TMA
  uint64_t* w_full = empty + p.stages;         // [1]       weights resident
  uint64_t* acc_full = w_full + 1;             // [nacc]    MMA -> epilogue
  uint64_t* acc_empty = acc_full + p.nacc;     // [nacc]    epilogue -> MMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + p.nacc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* red_run = reinterpret_cast<float*>(tmem_slot + 4);          // [epilogue warps][8 chunks][32 items]
  float* red_stat = red_run + kEpiWarps * 8 * 32;                    // mode 2: mean[Cn], invstd[Cn]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Start-up that needs nothing from global memory: it may run while the preceding kernel of the stream is
  // still at work (programmatic dependent launch, see elementwise.cuh).
  if (red.mode)
    for (int i = threadIdx.x; i < kEpiWarps * 8 * 32; i += kConvThreads) red_run[i] = 0.f;
  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_x)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_w)) : "memory");
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kConvMmaWarps); }
    mbar_init(w_full, 1);
    const int groups_per_tile = p.Cn / 16 < kEpiGroups ? p.Cn / 16 : kEpiGroups;
    for (int a = 0; a < p.nacc; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 4 * groups_per_tile); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(tmem_slot, p.tmem_cols);
  grid_dependency_wait();                  // from here on the preceding kernel's results may be read
  if (red.mode == 2)
    for (int i = threadIdx.x; i < 2 * p.Cn; i += kConvThreads) red_stat[i] = red.pstats[i];
  if (threadIdx.x == 0) {
    // This thread is also the producer: the weights and the first tile are requested now, so that their
    // latency runs beside the barrier below instead of after it.
    mbar_expect_tx(w_full, 9 * p.w_tx_bytes);
    for (int tap = 0; tap < 9; ++tap) tma_load_2d(w_smem + (size_t)tap * p.w_tap_bytes, &map_w, w_full, tap * p.Ck, 0);
    mbar_expect_tx(&full[0], p.tile_tx_bytes);
    tma_load_4d(smem, &map_x, &full[0], 0, -1, -1, (int)blockIdx.x * p.G);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int ksteps = p.Ck / 16;

  if (warp < kConvFirstEpiWarp) {
    if (lane == 0) {
      const uint32_t issuer = warp;                           // takes the 128-row tiles with acount % kConvMmaWarps == issuer
      // Issuer 0 is also the producer: before it starts on a tile it requests the tiles that fit into the free
      // stages (the weights and tile 0 were requested during set-up).  A stage's first use needs no wait; a
      // later one waits until every issuer has handed the stage back.
      uint32_t next_load = 1;
      // The tensors the epilogue reads row by row (residual, its gate, the two operands of a fused batch-norm
      // backward sum) are asked into L2 a whole tile ahead, so that the epilogue's loads do not wait for DRAM.
      auto prefetch_operands = [&](int tile) {
        int n0 = tile * p.G, n1 = n0 + p.G;
        if (n1 > p.N) n1 = p.N;
        const size_t img = (size_t)(p.sub == 1 ? p.H * p.W : (p.H >> 1) * (p.W >> 1)) * p.Cn;   // elements per image
        const size_t off = (size_t)n0 * img;
        const uint32_t bytes = (uint32_t)((size_t)(n1 - n0) * img * 2);
        if (res) prefetch_l2_bulk(res + off, bytes);
        if (res_mask) prefetch_l2_bulk(res_mask + off, bytes);
        if (red.mode == 2) { prefetch_l2_bulk(red.mask + off, bytes); prefetch_l2_bulk(red.xprev + off, bytes); }
      };
      if (issuer == 0) prefetch_operands((int)blockIdx.x);
      auto refill = [&](uint32_t upto) {
        if (issuer != 0) return true;
        for (; next_load < upto; ++next_load) {
          const int tile = (int)blockIdx.x + (int)next_load * (int)gridDim.x;
          if (tile >= p.tiles) return true;
          const int s = next_load % p.stages;
          const uint32_t ph = (next_load / p.stages) & 1;
          if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) return false;
          mbar_expect_tx(&full[s], p.tile_tx_bytes);
          tma_load_4d(smem + (size_t)s * p.stage_bytes, &map_x, &full[s], 0, -1, -1, tile * p.G);
          prefetch_operands(tile);
        }
        return true;
      };
      const uint32_t idesc = instr_desc(p.Cn, false);
      bool ok = mbar_wait(w_full, 0, abort_flag);
      tc_fence_after();
      // The issuing thread is the bottleneck when the instructions are this small, so the
      // descriptors are not rebuilt per instruction: a descriptor's low word holds the start
      // address in 16-byte units, and moving the operand is one 64-bit add.
      const uint64_t w_desc0 = smem_desc_kmajor(smem_u32(w_smem), p.pitch);
      const uint64_t w_tap_step = p.w_tap_bytes >> 4;
      uint64_t tap_off[9];                                   // operand shift of each filter tap, 16-byte units
#pragma unroll
      for (int tap = 0; tap < 9; ++tap) tap_off[tap] = (uint64_t)(((tap / 3) * p.Wp + (tap % 3)) * p.pitch) >> 4;
      const uint64_t mtile_step = (uint64_t)(kTileM * p.pitch) >> 4;
      // One tcgen05.mma of K = 16 occupies the tensor pipe for max(60, N/2) cycles whatever M is
      // and whether or not it depends on the previous one (measured), so a 128-row tile costs
      // 9 * Ck/16 * 60 cycles here and the only overhead worth removing is the issue loop's own.
      uint32_t it = 0, acount = 0;
      int slot = 0;                                           // acount % nacc and the slot's phase, kept incrementally
      uint32_t aph = 0;
      for (int tile = blockIdx.x; ok && tile < p.tiles && !*abort_flag; tile += gridDim.x, ++it) {
        if (!refill(it + (uint32_t)p.stages)) break;
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (!mbar_wait(&full[s], ph, abort_flag)) break;
        tc_fence_after();
        uint64_t x_desc = smem_desc_kmajor(smem_u32(smem + (size_t)s * p.stage_bytes), p.pitch);
        for (int i = 0; i < p.m_tiles; ++i, ++acount, x_desc += mtile_step) {
          if (acount % kConvMmaWarps == issuer) {
            if (acount >= (uint32_t)p.nacc) {                 // a slot's first use needs no hand-back from the epilogue
              if (!mbar_wait(&acc_empty[slot], aph ^ 1, abort_flag)) { ok = false; break; }
              tc_fence_after();
            }
            const uint32_t d_tmem = tmem_base + (uint32_t)slot * p.Cn;
            if (ksteps == 1) issue_tile<1>(d_tmem, x_desc, tap_off, w_desc0, w_tap_step, idesc);
            else if (ksteps == 2) issue_tile<2>(d_tmem, x_desc, tap_off, w_desc0, w_tap_step, idesc);
            else issue_tile<4>(d_tmem, x_desc, tap_off, w_desc0, w_tap_step, idesc);
            tc_commit(&acc_full[slot]);
          }
          if (++slot == p.nacc) { slot = 0; aph ^= 1; }
        }
        if (!ok) break;
        tc_commit(&empty[s]);
      }
    }
  } else {
    // Work item = (128-row tile, 16-column chunk), dealt to the groups in turn; the number of slots is
    // chosen (fwd_params) so that the same groups meet a slot every time and see all its phases.  The
    // global operands of an item (residual, its gate, the two tensors of a fused batch-norm-backward
    // sum) do not depend on the accumulator: they are requested one item ahead into the other of two
    // register sets, so that their latency runs beside the previous item's work.  Everything an item
    // needs (slot, phase, the pixel of this thread's row) is carried from item to item by additions:
    // a division per item costs more here than the item's arithmetic.
    const int lane_grp = warp & 3;                 // tensor-memory lanes 32*(warp % 4) .. +31
    const int group = (warp - kConvFirstEpiWarp) >> 2;
    const int nch = p.Cn >> 4;
    // Items are numbered J = (128-row tiles so far) * nch + chunk over the whole CTA; group g takes
    // J = g, g + kEpiGroups, ...  One step of J is `step_a` 128-row tiles and `step_c` chunks.
    const int step_a = kEpiGroups / nch, step_c = kEpiGroups - step_a * nch;
    struct Cursor {
      int tile, i;              // image tile, 128-row tile inside it
      int slot; uint32_t aph;   // accumulator slot of (tile, i) and the phase of its barriers
      int g, h, w;              // this thread's row of (tile, i) as (image in tile, padded row, padded column)
      int chunk; bool first_chunk;
    };
    struct Operands { bool valid; size_t base; uint4 r0, r1, g0, g1, k0, k1, x0, x1; };
    const int row0 = lane_grp * 32 + lane;
    const int g_first = row0 / p.img_rows, h_first = (row0 - g_first * p.img_rows) / p.Wp;
    const int w_first = row0 - g_first * p.img_rows - h_first * p.Wp;
    const int dh = kTileM / p.Wp, dw = kTileM - dh * p.Wp;            // 128 rows further on
    auto move_rows = [&](Cursor& c, int mtiles) {                     // this thread's row, `mtiles` 128-row tiles further on
      c.w += mtiles * dw; c.h += mtiles * dh;
      while (c.w >= p.Wp) { c.w -= p.Wp; ++c.h; }
      while (c.h >= p.Hp && c.g < p.G) { c.h -= p.Hp; ++c.g; }
    };
    auto move_mtiles = [&](Cursor& c, int da) {                       // da <= kEpiGroups <= nacc
      c.slot += da;
      if (c.slot >= p.nacc) { c.slot -= p.nacc; c.aph ^= 1; }
      c.i += da;
      if (c.i < p.m_tiles) { move_rows(c, da); return; }
      while (c.i >= p.m_tiles) { c.i -= p.m_tiles; c.tile += gridDim.x; }
      c.g = g_first; c.h = h_first; c.w = w_first;
      move_rows(c, c.i);
    };
    auto advance = [&](Cursor& c) -> bool {
      c.chunk += step_c;
      int da = step_a;
      if (c.chunk >= nch) { c.chunk -= nch; ++da; }
      c.first_chunk = da != 0;
      if (da) move_mtiles(c, da);
      return c.tile < p.tiles;
    };
    auto fetch = [&](const Cursor& c, Operands& o) {
      const int n = c.tile * p.G + c.g;
      o.valid = c.h < p.H && c.w < p.W && c.g < p.G && n < p.N && (p.sub == 1 || ((c.h | c.w) & 1) == 0);
      const int pix = p.sub == 1 ? (n * p.H + c.h) * p.W + c.w : (n * (p.H >> 1) + (c.h >> 1)) * (p.W >> 1) + (c.w >> 1);
      o.base = (size_t)pix * p.Cn + c.chunk * 16;
      if (red.mode == 2) o.k0 = o.k1 = o.x0 = o.x1 = make_uint4(0, 0, 0, 0);   // read below whether or not the row is valid
      if (!o.valid) return;
      if (res) {
        o.r0 = *reinterpret_cast<const uint4*>(res + o.base);
        o.r1 = *reinterpret_cast<const uint4*>(res + o.base + 8);
        if (res_mask) {
          o.g0 = *reinterpret_cast<const uint4*>(res_mask + o.base);
          o.g1 = *reinterpret_cast<const uint4*>(res_mask + o.base + 8);
        }
      }
      if (red.mode == 2) {
        o.k0 = *reinterpret_cast<const uint4*>(red.mask + o.base);
        o.k1 = *reinterpret_cast<const uint4*>(red.mask + o.base + 8);
        o.x0 = *reinterpret_cast<const uint4*>(red.xprev + o.base);
        o.x1 = *reinterpret_cast<const uint4*>(red.xprev + o.base + 8);
      }
    };
    // the group's first item: J = group
    Cursor cur{(int)blockIdx.x, 0, 0, 0u, g_first, h_first, w_first, 0, true};
    {
      const int a0 = group / nch;
      cur.chunk = group - a0 * nch;
      if (a0) move_mtiles(cur, a0);
    }
    // One item: request the next item's operands into `fill`, then finish the current one with `use`.
    // Returns false when there is no next item (or a wait gave up).
    auto item = [&](Operands& use, Operands& fill) -> bool {
      Cursor nxt = cur;
      const bool have_next = advance(nxt);
      if (have_next) fetch(nxt, fill);
      const int slot = cur.slot;
      if (cur.first_chunk) {
        if (!mbar_wait(&acc_full[slot], cur.aph, abort_flag)) return false;
        tc_fence_after();
      }
      const int c0 = cur.chunk * 16;
      uint32_t v[16];
      tmem_ld16(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)slot * p.Cn + c0, v);
      tmem_ld_wait();
      float f[16];
#pragma unroll
      for (int e = 0; e < 16; ++e) f[e] = __uint_as_float(v[e]);
      if (use.valid) {
        if (res) {
          const __nv_bfloat16* rb0 = reinterpret_cast<const __nv_bfloat16*>(&use.r0);
          const __nv_bfloat16* rb1 = reinterpret_cast<const __nv_bfloat16*>(&use.r1);
          float gq[16];
#pragma unroll
          for (int e = 0; e < 8; ++e) { gq[e] = __bfloat162float(rb0[e]); gq[8 + e] = __bfloat162float(rb1[e]); }
          if (res_mask) {
            const __nv_bfloat16* mb0 = reinterpret_cast<const __nv_bfloat16*>(&use.g0);
            const __nv_bfloat16* mb1 = reinterpret_cast<const __nv_bfloat16*>(&use.g1);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              if (!(__bfloat162float(mb0[e]) > 0.f)) gq[e] = 0.f;
              if (!(__bfloat162float(mb1[e]) > 0.f)) gq[8 + e] = 0.f;
            }
          }
#pragma unroll
          for (int e = 0; e < 16; ++e) f[e] += gq[e];
        }
        uint4 o0, o1;
        __nv_bfloat162* ob0 = reinterpret_cast<__nv_bfloat162*>(&o0);
        __nv_bfloat162* ob1 = reinterpret_cast<__nv_bfloat162*>(&o1);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          ob0[e] = __floats2bfloat162_rn(f[2 * e], f[2 * e + 1]);
          ob1[e] = __floats2bfloat162_rn(f[8 + 2 * e], f[8 + 2 * e + 1]);
        }
        *reinterpret_cast<uint4*>(out + use.base) = o0;
        *reinterpret_cast<uint4*>(out + use.base + 8) = o1;
      }
      if (red.mode) {
        float q[32];
        if (red.mode == 1) {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float sv = use.valid ? __bfloat162float(__float2bfloat16_rn(f[e])) : 0.f;
            q[e] = sv; q[16 + e] = sv * sv;
          }
        } else {
          const __nv_bfloat16* mb0 = reinterpret_cast<const __nv_bfloat16*>(&use.k0);
          const __nv_bfloat16* mb1 = reinterpret_cast<const __nv_bfloat16*>(&use.k1);
          const __nv_bfloat16* xb0 = reinterpret_cast<const __nv_bfloat16*>(&use.x0);
          const __nv_bfloat16* xb1 = reinterpret_cast<const __nv_bfloat16*>(&use.x1);
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float mk = __bfloat162float(e < 8 ? mb0[e] : mb1[e - 8]);
            const float xp = __bfloat162float(e < 8 ? xb0[e] : xb1[e - 8]);
            const float dz = (use.valid && mk > 0.f) ? __bfloat162float(__float2bfloat16_rn(f[e])) : 0.f;
            q[e] = dz;
            q[16 + e] = dz * ((xp - red_stat[c0 + e]) * red_stat[p.Cn + c0 + e]);
          }
        }
        transpose_reduce32(q, lane);
        red_run[((warp - kConvFirstEpiWarp) * 8 + (c0 >> 4)) * 32 + lane] += q[0];
      }
      if (!have_next || nxt.first_chunk) {           // this group's last chunk of the 128-row tile: hand the slot back
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[slot]);
      }
      cur = nxt;
      return have_next;
    };
    // 16-channel layers with batch-norm statistics and no residual (the forward convolutions of the first
    // stage, nine items per image): every item of a thread belongs to the same 16 channels, so the sums are
    // kept per thread and the lanes are combined once at the end; no global operands, no second register set.
    auto item_stats16 = [&](float (&run)[32]) -> bool {
      Cursor nxt = cur;
      const bool have_next = advance(nxt);
      const int n = cur.tile * p.G + cur.g;
      const bool valid = cur.h < p.H && cur.w < p.W && cur.g < p.G && n < p.N && (p.sub == 1 || ((cur.h | cur.w) & 1) == 0);
      const int pix = p.sub == 1 ? (n * p.H + cur.h) * p.W + cur.w : (n * (p.H >> 1) + (cur.h >> 1)) * (p.W >> 1) + (cur.w >> 1);
      const int slot = cur.slot;
      if (!mbar_wait(&acc_full[slot], cur.aph, abort_flag)) return false;
      tc_fence_after();
      uint32_t v[16];
      tmem_ld16(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)slot * p.Cn, v);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[slot]);            // the values are in registers: the slot is free
      if (valid) {
        uint4 o0, o1;
        __nv_bfloat162* ob0 = reinterpret_cast<__nv_bfloat162*>(&o0);
        __nv_bfloat162* ob1 = reinterpret_cast<__nv_bfloat162*>(&o1);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          ob0[e] = __floats2bfloat162_rn(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
          ob1[e] = __floats2bfloat162_rn(__uint_as_float(v[8 + 2 * e]), __uint_as_float(v[8 + 2 * e + 1]));
        }
        __nv_bfloat16* out_row = out + (size_t)pix * p.Cn;
        *reinterpret_cast<uint4*>(out_row) = o0;
        *reinterpret_cast<uint4*>(out_row + 8) = o1;
        const __nv_bfloat16* sb0 = reinterpret_cast<const __nv_bfloat16*>(&o0);
        const __nv_bfloat16* sb1 = reinterpret_cast<const __nv_bfloat16*>(&o1);
#pragma unroll
        for (int e = 0; e < 8; ++e) {                         // the statistics of the values as stored
          const float a = __bfloat162float(sb0[e]), b = __bfloat162float(sb1[e]);
          run[e] += a; run[16 + e] += a * a;
          run[8 + e] += b; run[24 + e] += b * b;
        }
      }
      cur = nxt;
      return have_next;
    };
    // The same for the data gradient that also forms the sums of the batch-norm backward it feeds
    // (no residual): the gate and the normalised tensor of an item are requested one item ahead.
    struct Operands2 { bool valid; int pix; uint4 k0, k1, x0, x1; };
    auto fetch2 = [&](const Cursor& c, Operands2& o) {
      const int n = c.tile * p.G + c.g;
      o.valid = c.h < p.H && c.w < p.W && c.g < p.G && n < p.N && (p.sub == 1 || ((c.h | c.w) & 1) == 0);
      o.pix = p.sub == 1 ? (n * p.H + c.h) * p.W + c.w : (n * (p.H >> 1) + (c.h >> 1)) * (p.W >> 1) + (c.w >> 1);
      o.k0 = o.k1 = o.x0 = o.x1 = make_uint4(0, 0, 0, 0);
      if (!o.valid) return;
      const size_t base = (size_t)o.pix * p.Cn;
      o.k0 = *reinterpret_cast<const uint4*>(red.mask + base);
      o.k1 = *reinterpret_cast<const uint4*>(red.mask + base + 8);
      o.x0 = *reinterpret_cast<const uint4*>(red.xprev + base);
      o.x1 = *reinterpret_cast<const uint4*>(red.xprev + base + 8);
    };
    auto item_bwd16 = [&](float (&run)[32], Operands2& use, Operands2& fill) -> bool {
      Cursor nxt = cur;
      const bool have_next = advance(nxt);
      if (have_next) fetch2(nxt, fill);
      const int slot = cur.slot;
      if (!mbar_wait(&acc_full[slot], cur.aph, abort_flag)) return false;
      tc_fence_after();
      uint32_t v[16];
      tmem_ld16(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)slot * p.Cn, v);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[slot]);
      if (use.valid) {
        uint4 o0, o1;
        __nv_bfloat162* ob0 = reinterpret_cast<__nv_bfloat162*>(&o0);
        __nv_bfloat162* ob1 = reinterpret_cast<__nv_bfloat162*>(&o1);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          ob0[e] = __floats2bfloat162_rn(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
          ob1[e] = __floats2bfloat162_rn(__uint_as_float(v[8 + 2 * e]), __uint_as_float(v[8 + 2 * e + 1]));
        }
        __nv_bfloat16* out_row = out + (size_t)use.pix * p.Cn;
        *reinterpret_cast<uint4*>(out_row) = o0;
        *reinterpret_cast<uint4*>(out_row + 8) = o1;
        const __nv_bfloat16* sb0 = reinterpret_cast<const __nv_bfloat16*>(&o0);
        const __nv_bfloat16* sb1 = reinterpret_cast<const __nv_bfloat16*>(&o1);
        const __nv_bfloat16* mb0 = reinterpret_cast<const __nv_bfloat16*>(&use.k0);
        const __nv_bfloat16* mb1 = reinterpret_cast<const __nv_bfloat16*>(&use.k1);
        const __nv_bfloat16* xb0 = reinterpret_cast<const __nv_bfloat16*>(&use.x0);
        const __nv_bfloat16* xb1 = reinterpret_cast<const __nv_bfloat16*>(&use.x1);
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float mk = __bfloat162float(e < 8 ? mb0[e] : mb1[e - 8]);
          const float xp = __bfloat162float(e < 8 ? xb0[e] : xb1[e - 8]);
          const float dz = mk > 0.f ? __bfloat162float(e < 8 ? sb0[e] : sb1[e - 8]) : 0.f;
          run[e] += dz;
          run[16 + e] += dz * ((xp - red_stat[e]) * red_stat[p.Cn + e]);
        }
      }
      cur = nxt;
      return have_next;
    };
    if (red.mode == 2 && nch == 1 && !res) {
      float run[32];
#pragma unroll
      for (int e = 0; e < 32; ++e) run[e] = 0.f;
      Operands2 oa, ob;
      if (!*abort_flag && cur.tile < p.tiles) {
        fetch2(cur, oa);
        while (item_bwd16(run, oa, ob) && item_bwd16(run, ob, oa)) {}
      }
      transpose_reduce32(run, lane);
      red_run[((warp - kConvFirstEpiWarp) * 8) * 32 + lane] += run[0];
    } else if (red.mode == 1 && nch == 1 && !res) {
      float run[32];
#pragma unroll
      for (int e = 0; e < 32; ++e) run[e] = 0.f;
      if (!*abort_flag && cur.tile < p.tiles) while (item_stats16(run)) {}
      transpose_reduce32(run, lane);
      red_run[((warp - kConvFirstEpiWarp) * 8) * 32 + lane] += run[0];
    } else {
      Operands op_a, op_b;
      if (!*abort_flag && cur.tile < p.tiles) {
        fetch(cur, op_a);
        while (item(op_a, op_b) && item(op_b, op_a)) {}
      }
    }
  }

  // Teardown.  After an abort, TMA copies may still be in flight towards this CTA's shared
  // memory: give every barrier that was armed a bounded chance to complete before leaving.
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) {
      if (error_word) atomicExch(error_word, 1);
      for (int s = 0; s <= p.stages; ++s) {
        uint64_t* b = s < p.stages ? &full[s] : w_full;
        for (uint32_t i = 0; i < (1u << 16); ++i)
          if (mbar_try_wait(b, 0) || mbar_try_wait(b, 1)) break;
      }
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
  if (red.mode && !*abort_flag) {
    // this CTA's sums: item (chunk, lane) of all epilogue warps, added in warp order -> partial[cta][stat][channel]
    const int pairs = 2 * p.Cn;
    for (int t = threadIdx.x; t < pairs; t += kConvThreads) {
      const int stat = t / p.Cn, c = t - stat * p.Cn;
      const int idx = (c >> 4) * 32 + (c & 15) + 16 * stat;
      float a = 0.f;
#pragma unroll
      for (int w = 0; w < kEpiWarps; ++w) a += red_run[w * 8 * 32 + idx];
      red.partial[(size_t)blockIdx.x * pairs + t] = a;
    }
  }
}

// ------------------------------------------------------------- weight gradient --
// With q' = q + r*Wp the sum becomes dW[n][r][s][c] = sum_q' dY[q' - r*Wp][n] * X[q' + s][c], so ONE
// instruction per 16-pixel step covers all nine taps: the A operand stacks the taps s of a filter
// row along M (M-blocks one pixel apart in the x tile), the B operand stacks the filter rows along
// N (N-blocks Wp pixels apart in the dy tile, which is loaded with two extra zero rows on top so
// that block b = 2 - r starts at row q' + b*Wp).  N = 3*Co <= 192 costs the same 60..96 cycles as
// N = Co would.
struct WgradParams {
  int W, H, N, Wp, Hp;
  int Ci, Co;                 // channels of x and of dy
  int kcx, kcy;               // channel chunk of the x and of the dy tile (16/32/64): a CTA computes the block
  int nyb;                    //   dW[co chunk b][.][.][ci chunk a], blockIdx.y = a * nyb + b
  int G, tiles;               // images per tile, ceil(N / G)
  int ksteps;                 // 16-pixel reduction steps per tile
  uint32_t pitch_x, pitch_y;
  uint32_t x_tx_bytes, y_tx_bytes;
  uint32_t x_bytes, y_bytes;  // shared memory reserved per stage for the two tiles (multiples of 1024)
  int stages;
  int sgroups;                // M-block groups: 1, or 2 when kcx = 64 (128 rows hold only two taps)
  int taps_per_group;         // min(3, 128 / kcx)
  uint32_t tmem_cols;
};

__global__ void __launch_bounds__(kFwdThreads, 1)
wgrad_halo_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y, WgradParams p,
                  float* __restrict__ partial, int* __restrict__ error_word) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t stage_bytes = p.x_bytes + p.y_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)p.stages * stage_bytes);
  uint64_t* full = bars;
  uint64_t* empty = full + p.stages;
  uint64_t* done = empty + p.stages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(done + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk_a = blockIdx.y / p.nyb, chunk_b = blockIdx.y - chunk_a * p.nyb;
  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_x)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_y)) : "memory");
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kMmaWarps); }
    mbar_init(done, kMmaWarps);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // the producer's first pair of tiles, requested during set-up (they do not touch the slack cleared below)
    mbar_expect_tx(&full[0], p.x_tx_bytes + p.y_tx_bytes);
    tma_load_4d(smem, &map_x, &full[0], chunk_a * p.kcx, -1, -1, (int)blockIdx.x * p.G);
    tma_load_4d(smem + p.x_bytes, &map_y, &full[0], chunk_b * p.kcy, 0, -2, (int)blockIdx.x * p.G);
  }
  // The reduction runs over whole 16-pixel steps and the stacked blocks read some pixels past
  // the tile: that slack is never written by TMA, so it is cleared once (a stray NaN there
  // would survive the multiplication by a zero of the other operand).
  for (int s = 0; s < p.stages; ++s) {
    uint8_t* xs = smem + (size_t)s * stage_bytes;
    uint8_t* ys = xs + p.x_bytes;
    for (uint32_t o = p.x_tx_bytes + threadIdx.x * 16; o < p.x_bytes; o += kFwdThreads * 16) *reinterpret_cast<uint4*>(xs + o) = make_uint4(0, 0, 0, 0);
    for (uint32_t o = p.y_tx_bytes + threadIdx.x * 16; o < p.y_bytes; o += kFwdThreads * 16) *reinterpret_cast<uint4*>(ys + o) = make_uint4(0, 0, 0, 0);
  }
  fence_proxy_async();
  if (warp == 1) tmem_alloc(tmem_slot, p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int ncols = 3 * p.kcy;                                // N of the instruction

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 1;                                        // the first pair was requested during set-up
      for (int tile = blockIdx.x + gridDim.x; tile < p.tiles && !*abort_flag; tile += gridDim.x, ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) break;
        uint8_t* xs = smem + (size_t)s * stage_bytes;
        mbar_expect_tx(&full[s], p.x_tx_bytes + p.y_tx_bytes);
        tma_load_4d(xs, &map_x, &full[s], chunk_a * p.kcx, -1, -1, tile * p.G);
        tma_load_4d(xs + p.x_bytes, &map_y, &full[s], chunk_b * p.kcy, 0, -2, tile * p.G);
      }
    }
  } else if (warp < kFirstEpiWarp) {
    if (lane == 0) {
      // Two issuing warps.  One tap group (Ci <= 32): the reduction steps alternate between them, each
      // into its own copy of the accumulator (the epilogue adds the two).  Two tap groups: one each.
      const uint32_t issuer = warp - 1;
      const uint32_t idesc = instr_desc(ncols, true);
      const uint64_t a_kstep = (uint64_t)(16 * p.pitch_x) >> 4, b_kstep = (uint64_t)(16 * p.pitch_y) >> 4;
      const uint64_t a_group = (uint64_t)(p.taps_per_group * p.pitch_x) >> 4;
      const uint32_t d_tmem = tmem_base + issuer * (uint32_t)ncols;
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.tiles && !*abort_flag; tile += gridDim.x, ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (!mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t x_addr = smem_u32(smem + (size_t)s * stage_bytes);
        uint64_t a_desc = smem_desc_mnmajor(x_addr, p.pitch_x, p.pitch_x);
        uint64_t b_desc = smem_desc_mnmajor(x_addr + p.x_bytes, p.pitch_y, (uint32_t)p.Wp * p.pitch_y);
        if (p.sgroups == 1) {
          a_desc += issuer * a_kstep; b_desc += issuer * b_kstep;
          for (int j = (int)issuer; j < p.ksteps; j += kMmaWarps, a_desc += kMmaWarps * a_kstep, b_desc += kMmaWarps * b_kstep)
            tc_mma_bf16(d_tmem, a_desc, b_desc, idesc, it != 0 || j >= kMmaWarps);
        } else {
          a_desc += issuer * a_group;
          for (int j = 0; j < p.ksteps; ++j, a_desc += a_kstep, b_desc += b_kstep)
            tc_mma_bf16(d_tmem, a_desc, b_desc, idesc, (it | (uint32_t)j) != 0);
        }
        tc_commit(&empty[s]);
      }
      if (ok) tc_commit(done);
    }
  } else {
    // kEpiGroups groups of four warps share the write-out: the (tap group, 16-column chunk)
    // items are dealt to the groups in turn.
    const int lane_grp = warp & 3;
    const int group = (warp - kFirstEpiWarp) >> 2;
    if (mbar_wait(done, 0, abort_flag)) {
      tc_fence_after();
      const int row = lane_grp * 32 + lane;
      const int sblk = row / p.kcx, ci = chunk_a * p.kcx + (row - sblk * p.kcx);
      float* dst = partial + (size_t)blockIdx.x * ((size_t)p.Co * 9 * p.Ci);
      const int nchunks = ncols >> 4;
      const size_t co_stride = (size_t)9 * p.Ci;
      for (int item = group; item < p.sgroups * nchunks; item += kEpiGroups) {
        const int sg = item / nchunks, c0 = (item - sg * nchunks) << 4;
        const int sx = sg * p.taps_per_group + sblk;
        const bool valid = sblk < p.taps_per_group && sx < 3;
        uint32_t v[16];
        tmem_ld16(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(sg * ncols + c0), v);
        tmem_ld_wait();
        if (p.sgroups == 1) {                     // the second issuer's copy of the accumulator
          uint32_t u[16];
          tmem_ld16(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(ncols + c0), u);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 16; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) + __uint_as_float(u[e]));
        }
        if (!valid) continue;
        const int b = c0 / p.kcy, r = 2 - b, co0 = chunk_b * p.kcy + (c0 - b * p.kcy);   // kcy is a multiple of 16: a chunk stays in one block
        float* d0 = dst + (size_t)co0 * co_stride + (size_t)(r * 3 + sx) * p.Ci + ci;
#pragma unroll
        for (int e = 0; e < 16; ++e) d0[(size_t)e * co_stride] = __uint_as_float(v[e]);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) {
      if (error_word) atomicExch(error_word, 1);
      for (int s = 0; s < p.stages; ++s)
        for (uint32_t i = 0; i < (1u << 16); ++i)
          if (mbar_try_wait(&full[s], 0) || mbar_try_wait(&full[s], 1)) break;
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

// dw[i] = sum over the pixel-split CTAs of partial[cta][i], in CTA order.  A block owns 32
// consecutive outputs; its 8 warps take interleaved CTAs and are added in warp order.
__global__ void __launch_bounds__(256) wgrad_halo_reduce_kernel(const float* __restrict__ partial, float* __restrict__ dw, size_t n, int ctas) {
  __shared__ float part[8][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const size_t i = (size_t)blockIdx.x * 32 + lane;
  float a = 0.f;
  if (i < n)
    for (int z = warp; z < ctas; z += 8) a += partial[(size_t)z * n + i];
  part[warp][lane] = a;
  __syncthreads();
  if (warp == 0 && i < n) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) t += part[w][lane];
    dw[i] = t;
  }
}

// ----------------------------------------------------------------- host side ---
inline uint32_t round_up_u32(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }
constexpr size_t kSmemBudget = 200 * 1024;

constexpr size_t kFixedSmem = kRedSmemBytes + 4096;      // reduction scratch, barriers, alignment slack
inline bool chan_ok(int c) { return c == 16 || c == 32 || c == 64; }

inline FwdParams fwd_params(int N, int H, int W, int Ck, int Cn, int sm_count) {
  FwdParams p{};
  p.W = W; p.H = H; p.N = N; p.Wp = W + 2; p.Hp = H + 2; p.Ck = Ck; p.Cn = Cn;
  p.sub = 1;
  p.img_rows = p.Hp * p.Wp;
  p.pitch = (uint32_t)Ck * 2;
  p.w_tx_bytes = (uint32_t)Cn * p.pitch;
  p.w_tap_bytes = round_up_u32(p.w_tx_bytes, 1024);
  // images per tile: as many as keep every SM busy, within the shared-memory budget
  int G = N / 148;                                            // more than one image per tile only for large batches
  if (G < 1) G = 1;
  for (;; --G) {
    p.G = G;
    p.m_tiles = (((G - 1) * p.Hp + (H - 1)) * p.Wp + W + kTileM - 1) / kTileM;
    uint32_t rows = (uint32_t)(kTileM * p.m_tiles + 2 * p.Wp + 2);
    if (rows < (uint32_t)(G * p.img_rows)) rows = (uint32_t)(G * p.img_rows);
    p.stage_bytes = round_up_u32(rows * p.pitch, 1024);
    if (G == 1 || 2 * (size_t)p.stage_bytes + 9 * (size_t)p.w_tap_bytes + kFixedSmem <= kSmemBudget) break;
  }
  p.tiles = (N + p.G - 1) / p.G;
  p.tile_tx_bytes = (uint32_t)(p.G * p.img_rows) * p.pitch;
  const size_t fixed = 9 * (size_t)p.w_tap_bytes + kFixedSmem;
  int stages = fixed < kSmemBudget ? (int)((kSmemBudget - fixed) / p.stage_bytes) : 0;
  const int per_cta = (p.tiles + (sm_count > 0 ? sm_count : 148) - 1) / (sm_count > 0 ? sm_count : 148);
  if (stages > 3) stages = 3;
  if (stages > per_cta) stages = per_cta;                     // shared memory left free lets other kernels' CTAs co-reside
  p.stages = stages;
  // Accumulator slots.  Two conditions keep every waiter in step with the phases of a slot's barriers:
  // an even count, so that a slot always belongs to the same issuing warp (the warps take alternate
  // 128-row tiles); and, where a tile has fewer chunks than there are epilogue groups, a count whose
  // chunk total is a multiple of the groups, so that the same groups meet a slot every time.  Within
  // that, a slot per 128-row tile where 256 columns allow it, so the issuers seldom wait for the epilogue.
  {
    const int nch = Cn / 16;
    int step = kConvMmaWarps;
    if (nch < kEpiGroups) {
      int g = kEpiGroups, a = nch;                           // kEpiGroups / gcd(kEpiGroups, nch)
      while (a) { const int t = g % a; g = a; a = t; }
      const int need = kEpiGroups / g;
      step = need % kConvMmaWarps == 0 ? need : need * kConvMmaWarps;
    }
    p.nacc = (p.m_tiles + step - 1) / step * step;
    while (p.nacc > step && p.nacc * Cn > 256) p.nacc -= step;
  }
  uint32_t cols = 32;
  while (cols < (uint32_t)(p.nacc * Cn)) cols <<= 1;
  p.tmem_cols = cols;
  return p;
}

inline size_t fwd_smem_bytes(const FwdParams& p) {
  return (size_t)p.stages * p.stage_bytes + 9 * (size_t)p.w_tap_bytes + (size_t)(2 * p.stages + 1 + 2 * p.nacc) * 8 + 16 +
         kRedSmemBytes + 1024;
}

inline bool fwd_supported(int N, int H, int W, int Ck, int Cn) {
  if (!chan_ok(Ck) || Cn % 16 || Cn < 16 || Cn > 128) return false;
  if (W + 2 > 256 || H + 2 > 256 || N < 1) return false;
  FwdParams p = fwd_params(N, H, W, Ck, Cn, 148);
  return p.stages >= 1 && fwd_smem_bytes(p) <= kSmemBudget + 4096 && p.tile_tx_bytes < (1u << 20) && p.tmem_cols <= 512;
}

// Channel chunk of a tile: the whole pixel when it is one swizzle span, else 64- or 32-channel slices.
inline int wgrad_chunk(int C) { return chan_ok(C) ? C : (C % 64 == 0 ? 64 : (C % 32 == 0 ? 32 : 0)); }

inline WgradParams wgrad_params(int N, int H, int W, int Ci, int Co) {
  WgradParams p{};
  p.W = W; p.H = H; p.N = N; p.Wp = W + 2; p.Hp = H + 2; p.Ci = Ci; p.Co = Co;
  p.kcx = wgrad_chunk(Ci); p.kcy = wgrad_chunk(Co);
  if (p.kcx == 0 || p.kcy == 0) { p.stages = 0; return p; }
  p.nyb = Co / p.kcy;
  p.pitch_x = (uint32_t)p.kcx * 2; p.pitch_y = (uint32_t)p.kcy * 2;
  const int img_rows = p.Hp * p.Wp;
  // images per tile: what two pipeline stages of both tiles fit in shared memory
  const int max_rows = (int)(96 * 1024 / (p.pitch_x + p.pitch_y));
  p.G = max_rows / img_rows > 0 ? max_rows / img_rows : 1;
  if (p.G > N) p.G = N;
  p.tiles = (N + p.G - 1) / p.G;
  const int Q = p.G * img_rows;
  p.ksteps = (Q + 15) / 16;
  const int blocks = kTileM / p.kcx;
  p.taps_per_group = blocks < 3 ? blocks : 3;
  p.sgroups = (3 + p.taps_per_group - 1) / p.taps_per_group;
  p.x_tx_bytes = (uint32_t)Q * p.pitch_x; p.y_tx_bytes = (uint32_t)Q * p.pitch_y;
  p.x_bytes = round_up_u32((uint32_t)(16 * p.ksteps + 2 * blocks + 16) * p.pitch_x, 1024);
  p.y_bytes = round_up_u32((uint32_t)(16 * p.ksteps + 2 * p.Wp + 16) * p.pitch_y, 1024);
  const size_t stage = (size_t)p.x_bytes + p.y_bytes;
  int stages = (int)((kSmemBudget - 2048) / stage);
  p.stages = stages > 2 ? 2 : stages;
  uint32_t need = (uint32_t)(2 * 3 * p.kcy), cols = 32;         // two accumulators: two tap groups, or two copies of one
  while (cols < need) cols <<= 1;
  p.tmem_cols = cols;
  return p;
}
inline int wgrad_pairs(const WgradParams& p) { return (p.Ci / p.kcx) * (p.Co / p.kcy); }

// Pixel split: few enough CTAs that their partial sums (Co*9*Ci floats each) stay small next to
// the operands, enough of them to spread the reduction over the SMs.  `cap` (0 = none) bounds the
// split further: beside other kernels a weight gradient that is nobody's next input does better on
// a few SMs for longer than on many at once (measured: 16 CTAs instead of 64-128 take 9 % off an
// iteration of four concurrent modules).  Scratch is sized for cap = 0.
inline int wgrad_ctas(const WgradParams& p, int cap = 0) {
  const int pairs = wgrad_pairs(p);
  int want;
  if (pairs > 1) {                                              // chunked (wide) layers: about 1.5 CTAs per SM in all
    want = (222 + pairs / 2) / pairs;
    if (cap > 0 && want * pairs > 4 * cap) want = 4 * cap / pairs;
  } else {
    const size_t wsize = (size_t)p.Co * 9 * p.Ci;
    want = (int)((size_t)p.N * p.H * p.W * (p.Ci + p.Co) * 2 / (wsize * 2));     // partial bytes <= ~ 2 x operand bytes
    if (want > 128) want = 128;
    if (want < 32) want = 32;
    if (cap > 0 && want > cap) want = cap;
  }
  if (want < 1) want = 1;
  return p.tiles < want ? p.tiles : want;
}
inline size_t wgrad_smem_bytes(const WgradParams& p) {
  return (size_t)p.stages * ((size_t)p.x_bytes + p.y_bytes) + (size_t)(2 * p.stages + 1) * 8 + 16 + 1024;
}
inline bool wgrad_supported(int N, int H, int W, int Ci, int Co) {
  if (wgrad_chunk(Ci) == 0 || wgrad_chunk(Co) == 0) return false;
  if (W + 2 > 256 || H + 2 > 256 || N < 1) return false;
  WgradParams p = wgrad_params(N, H, W, Ci, Co);
  return p.stages >= 1 && p.x_tx_bytes < (1u << 19) && p.y_tx_bytes < (1u << 19) && p.tmem_cols <= 512 &&
         wgrad_pairs(p) <= 65535;
}
// fp32 elements of scratch the weight gradient needs for its per-CTA partial sums.
inline size_t wgrad_scratch_elems(int N, int H, int W, int Ci, int Co) {
  WgradParams p = wgrad_params(N, H, W, Ci, Co);
  return (size_t)wgrad_ctas(p) * Co * 9 * Ci;
}

// Halo-tile tensor map of a bf16 NHWC tensor: box = G whole images with border.
inline cudaError_t make_tile_map(const void* act, int N, int H, int W, int C, int G, CUtensorMap* map, int boxC = 0) {
  if (boxC == 0) boxC = C;
  EncodeTiledFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
  cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
  cuuint32_t box[4] = {(cuuint32_t)boxC, (cuuint32_t)(W + 2), (cuuint32_t)(H + 2), (cuuint32_t)G};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  if (enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(act), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(boxC * 2), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  return cudaSuccess;
}
// Weight map: bf16 [Cn][9*Ck], box = one filter tap of all Cn rows.
inline cudaError_t make_weight_map(const void* wgt, int Ck, int Cn, CUtensorMap* map) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  cuuint64_t dims[2] = {(cuuint64_t)9 * Ck, (cuuint64_t)Cn};
  cuuint64_t strides[1] = {(cuuint64_t)9 * Ck * 2};
  cuuint32_t box[2] = {(cuuint32_t)Ck, (cuuint32_t)Cn};
  cuuint32_t estr[2] = {1, 1};
  if (enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(wgt), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(Ck * 2), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  return cudaSuccess;
}

inline cudaError_t set_smem_attrs() {
  static bool done = false;
  if (done) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(conv_halo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget + 8192);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(wgrad_halo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget + 8192);
  if (e == cudaSuccess) done = true;
  return e;
}

}  // namespace halo
}  // namespace fdg
