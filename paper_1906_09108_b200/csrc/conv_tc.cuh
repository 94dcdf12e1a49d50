// 3x3 / stride 1 / pad 1 convolution forward and data gradient as an implicit GEMM on the
// sm_100a tensor cores: bf16 operands staged in shared memory by TMA, tcgen05.mma with fp32
// accumulators in tensor memory, epilogue through tcgen05.ld.
//
//   D[m][n] = sum_{tap, c} A_tap[m][c] * B_tap[n][c]
//     m   = 128 consecutive output pixels: whole image rows (or whole images) of an NHWC tensor
//     A   = the input shifted by the tap offset; the TMA box starts at (w-1+s, h-1+r) and the
//           hardware zero-fills what falls outside the image, which is the padding
//     B   = weights [N][9*C]: forward [c_out][r][s][c_in]; data gradient: the flipped and
//           transposed copy [c_in][2-r][2-s][c_out] (dgrad of a stride-1 3x3 conv is a 3x3 conv)
//   Both operands are K-major with the channel chunk (16/32/64 channels = 32/64/128 bytes) as
//   the swizzle span, so the TMA swizzle mode and the MMA descriptor layout agree.
//
// One persistent CTA per SM walks tiles (m-tile, n-tile); roles by warp:
//   warp 0      TMA producer: per (tap, channel chunk) one A box and one B box into a ring stage
//   warp 1      MMA issuer: C_chunk/16 tcgen05.mma per stage, tcgen05.commit frees the stage;
//               after the last stage of a tile a commit hands the accumulator to the epilogue
//   warps 2..5  epilogue: TMEM -> registers -> (+ residual) -> bf16 -> global, 32 rows per warp
// Two accumulators alternate so the epilogue of tile i overlaps the MMAs of tile i+1.
// Every wait is bounded: on time-out the CTA raises an error word and leaves without hanging.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace fdg {
namespace tc {

constexpr int kTileM = 128;
constexpr int kThreads = 192;            // 6 warps
constexpr uint32_t kSpinLimit = 1u << 24;

struct ConvTcParams {
  int W, H, N;              // image width, height, batch
  int rows_per_tile;        // image rows per tile when a tile stays inside one image, else H
  int imgs_per_tile;        // images per tile (1 unless 128 pixels span whole images)
  int Ci, Co;               // GEMM-K channels per tap, GEMM-N total
  int kc;                   // channel chunk per stage: 16, 32 or 64
  int n_tile;               // GEMM-N per tile (multiple of 16, <= 256)
  int m_tiles, n_tiles;
  int stages;
  uint32_t a_bytes, b_bytes, stage_bytes;   // b_bytes is padded to 1 KiB; b_tx_bytes is what TMA moves
  uint32_t b_tx_bytes;
  uint32_t tmem_cols;       // allocated columns (power of two >= 2*n_tile)
  int mpair;                // 128-row tiles a CTA works on at once with one weight tile: 1 (two accumulator sets, the
                            // epilogue of a tile overlaps the next tile's instructions) or 2 (one set of two accumulators:
                            // every weight tile fetched from L2 serves 256 rows)
  int sub;                  // 1, or 2: store only the pixels with even h and w, as an [N][H/2][W/2][Co] tensor,
                            // or 3: store pixel (h, w) at (2h, 2w) of an [N][2H][2W][Co] tensor (the data gradient of a
                            // stride-2 1x1 convolution; the other pixels of that tensor are not touched)
  int taps;                 // 9 (3x3, pad 1) or 1 (1x1, pad 0)
  int act_sub;              // 1, or 2: the activation operand is the even pixels of an [N][2H][2W][Ci] tensor
  int patch;                // 1: conv3x3_patch_kernel (16x16-pixel patches with their halo), 0: conv3x3_tc_kernel
  uint32_t halo_bytes;      // patch mode: shared memory of one 18x18-pixel halo tile of kc channels (multiple of 1 KiB)
  int b_stages;             // patch mode: weight tiles in flight
  int acc_slots;            // patch mode: accumulators of n_tile columns the 128-row tiles rotate over (3 where tensor
                            // memory holds them: the write-out of a tile then runs beside the next tiles' instructions)
};
constexpr int kPatch = 16;                         // patch side in pixels
constexpr int kPatchHalo = kPatch + 2;             // with the one-pixel border

// ---------------------------------------------------------------- PTX wrappers --
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false when the limit is hit or another role has raised *abort_flag.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t limit = kSpinLimit) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023) == 1023 && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

// One warp waits, with the bounded wait above, on a barrier that nothing ever arrives at: after `limit`
// polls the wait gives up and the kernel reports it the way the convolution kernels do.  Nothing is in
// flight and no tensor memory is held when it leaves.  Lets the host-side handling of a wait that ran
// out be exercised without making a real kernel misbehave.
__global__ void wait_probe_kernel(uint32_t limit, int* error_word) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int flag;
  volatile int* abort_flag = &flag;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait(&bar, 0, abort_flag, limit);
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0 && error_word) atomicExch(error_word, 1);
}

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, K-major operand whose rows are one swizzle span wide:
// rows of `row_bytes` (32/64/128), 8-row groups `8*row_bytes` apart.
__device__ __forceinline__ uint64_t smem_desc_kmajor(uint32_t addr, uint32_t row_bytes) {
  const uint64_t layout = row_bytes == 128 ? 2 : (row_bytes == 64 ? 4 : 6);   // SWIZZLE_128B / 64B / 32B
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);                 // start address, 16-byte units
  d |= (uint64_t)1 << 16;                                // leading byte offset (unused for one span)
  d |= (uint64_t)(((8 * row_bytes) >> 4) & 0x3FFF) << 32;   // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                                // descriptor version of this architecture
  d |= layout << 61;
  return d;
}
// The same with an explicit distance between 8-row groups (rows inside a group stay one span apart).
__device__ __forceinline__ uint64_t smem_desc_kmajor_sbo(uint32_t addr, uint32_t row_bytes, uint32_t group_bytes) {
  const uint64_t layout = row_bytes == 128 ? 2 : (row_bytes == 64 ? 4 : 6);
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)((group_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= layout << 61;
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128.
__device__ __forceinline__ uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}

// 32 lanes each hold 32 items; afterwards lane l holds in q[0] the sum over all lanes of item l.
__device__ __forceinline__ void transpose_reduce32(float (&q)[32], int lane) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    const bool upper = (lane & off) != 0;
#pragma unroll
    for (int i = 0; i < off; ++i) {
      const float send = upper ? q[i] : q[i + off];
      const float keep = upper ? q[i + off] : q[i];
      q[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
}

// Batch-norm statistics of the output, formed in the epilogue (optional): every epilogue warp adds, per 16-channel
// chunk, the sums of the values it stores and of their squares over its 32 rows into its own array in shared
// memory; at the end the CTA writes one row stat_partial[blockIdx.x][2][Co] (sum, sum of squares), which
// stats_finalize_kernel adds over the CTAs in CTA order.  Up to kStatChunks * 16 output channels.
constexpr int kStatChunks = 40;
constexpr int kStatFloats = 4 * kStatChunks * 32;
__device__ __forceinline__ void stat_add(float* stat_run, int ew, int chunk, const uint4& o0, const uint4& o1, int lane) {
  const __nv_bfloat16* sb0 = reinterpret_cast<const __nv_bfloat16*>(&o0);
  const __nv_bfloat16* sb1 = reinterpret_cast<const __nv_bfloat16*>(&o1);
  float q[32];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const float a = __bfloat162float(sb0[e]), b = __bfloat162float(sb1[e]);      // the values as stored
    q[e] = a; q[8 + e] = b; q[16 + e] = a * a; q[24 + e] = b * b;
  }
  transpose_reduce32(q, lane);
  stat_run[(ew * kStatChunks + chunk) * 32 + lane] += q[0];
}
// The CTA's row of partial sums (after all epilogue warps are done).
__device__ __forceinline__ void stat_flush(const float* stat_run, float* __restrict__ stat_partial, int Co) {
  for (int t = threadIdx.x; t < 2 * Co; t += blockDim.x) {
    const int stat = t / Co, c = t - stat * Co;
    const int idx = (c >> 4) * 32 + (c & 15) + 16 * stat;
    float a = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) a += stat_run[w * kStatChunks * 32 + idx];
    stat_partial[(size_t)blockIdx.x * 2 * Co + t] = a;
  }
}

// ------------------------------------------------------------------- kernel ----
// out[m][n] (bf16, row stride Co) = conv + (res ? res[m][n] * [mask ? mask[m][n] > 0 : 1] : 0)
__global__ void __launch_bounds__(kThreads, 1)
conv3x3_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  ConvTcParams p, __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ res,
                  const __nv_bfloat16* __restrict__ res_mask, float* __restrict__ stat_partial, int* __restrict__ error_word) {
  __shared__ float stat_run[kStatFloats];
  if (stat_partial) for (int i = threadIdx.x; i < kStatFloats; i += blockDim.x) stat_run[i] = 0.f;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)p.stages * p.stage_bytes);
  uint64_t* full = bars;                       // [stages]  TMA -> MMA
  uint64_t* empty = bars + p.stages;           // [stages]  MMA -> TMA
  uint64_t* acc_full = empty + p.stages;       // [2]       MMA -> epilogue
  uint64_t* acc_empty = acc_full + 2;          // [2]       epilogue -> MMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(tmem_slot, p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int chunks = (p.Ci + p.kc - 1) / p.kc;
  const int k_iters = p.taps * chunks;
  const int total_tiles = ((p.m_tiles + p.mpair - 1) / p.mpair) * p.n_tiles;     // tiles of mpair * 128 rows

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      for (int tile = blockIdx.x; tile < total_tiles && !*abort_flag; tile += gridDim.x) {
        const int mg = tile / p.n_tiles, nt = tile - mg * p.n_tiles;
        int n0[2], h0[2];
        const int halves = (mg * p.mpair + 1 < p.m_tiles) ? p.mpair : 1;
        for (int hf = 0; hf < halves; ++hf) {
          const int mt = mg * p.mpair + hf;
          if (p.imgs_per_tile == 1) {
            const int tiles_per_img = p.H / p.rows_per_tile;
            n0[hf] = mt / tiles_per_img; h0[hf] = (mt - n0[hf] * tiles_per_img) * p.rows_per_tile;
          } else {
            n0[hf] = mt * p.imgs_per_tile; h0[hf] = 0;
          }
        }
        for (int ki = 0; ki < k_iters; ++ki, ++it) {
          const int s = it % p.stages;
          const uint32_t ph = (it / p.stages) & 1;
          if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) break;
          const int tap = ki / chunks, cc = ki - tap * chunks;
          const int r = tap / 3, sx = tap - r * 3;
          const int dw = p.taps == 1 ? 0 : sx - 1, dh = p.taps == 1 ? 0 : r - 1;
          uint8_t* a_dst = smem + (size_t)s * p.stage_bytes;
          uint8_t* b_dst = a_dst + (size_t)p.mpair * p.a_bytes;
          mbar_expect_tx(&full[s], (uint32_t)halves * p.a_bytes + p.b_tx_bytes);
          for (int hf = 0; hf < halves; ++hf)
            tma_load_4d(a_dst + (size_t)hf * p.a_bytes, &map_a, &full[s], cc * p.kc, dw, h0[hf] + dh, n0[hf]);
          tma_load_2d(b_dst, &map_b, &full[s], tap * p.Ci + cc * p.kc, nt * p.n_tile);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(p.n_tile);
      const uint32_t row_bytes = p.kc * 2;
      uint32_t it = 0, tcount = 0;
      const int nsets = p.mpair == 1 ? 2 : 1;                  // accumulator sets in tensor memory
      // Descriptors are formed once per stage; moving an operand is a 64-bit add on the address field (the issuing
      // thread is alone in its warp, so every instruction between two tcgen05.mma costs its full latency).
      uint64_t a_desc[8], b_desc[8];
      for (int i = 0; i < 8; ++i) {
        const uint32_t a_addr = smem_u32(smem + (size_t)(i < p.stages ? i : 0) * p.stage_bytes);
        a_desc[i] = smem_desc_kmajor(a_addr, row_bytes);
        b_desc[i] = smem_desc_kmajor(a_addr + (uint32_t)p.mpair * p.a_bytes, row_bytes);
      }
      const uint64_t half_off = (uint64_t)p.a_bytes >> 4;
      const int ksub = p.kc / 16;
      int s = 0;
      uint32_t ph = 0;                                         // it % stages and that stage's phase, kept incrementally
      for (int tile = blockIdx.x; tile < total_tiles && !*abort_flag; tile += gridDim.x, ++tcount) {
        const int acc = (int)(tcount % nsets);
        const uint32_t acc_ph = (tcount / nsets) & 1;
        if (!mbar_wait(&acc_empty[acc], acc_ph ^ 1, abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * p.n_tile;
        const int mg = tile / p.n_tiles;
        const int halves = (mg * p.mpair + 1 < p.m_tiles) ? p.mpair : 1;
        bool ok = true;
        for (int ki = 0; ki < k_iters; ++ki, ++it) {
          if (!mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t a0 = a_desc[s], b0 = b_desc[s];
          // Straight-line issue: the choice between one and two 128-row tiles is made outside the loop over the
          // K steps (a branch between two tcgen05.mma costs the lone issuing thread tens of cycles, see
          // mma_rate_kernel), and the two tiles take turns.
          if (halves == 2) {
            for (int j = 0; j < ksub; ++j) {
              tc_mma_bf16(d_tmem, a0 + 2 * j, b0 + 2 * j, idesc, (ki | j) != 0);
              tc_mma_bf16(d_tmem + (uint32_t)p.n_tile, a0 + half_off + 2 * j, b0 + 2 * j, idesc, (ki | j) != 0);
            }
          } else {
            for (int j = 0; j < ksub; ++j) tc_mma_bf16(d_tmem, a0 + 2 * j, b0 + 2 * j, idesc, (ki | j) != 0);
          }
          tc_commit(&empty[s]);
          if (++s == p.stages) { s = 0; ph ^= 1; }
        }
        if (!ok) break;
        tc_commit(&acc_full[acc]);
      }
    }
  } else {
    const int ew = warp - 2;                       // TMEM lanes 32*(warp%4) belong to this warp
    const int lane_grp = warp & 3;
    (void)ew;
    uint32_t tcount = 0;
    const int nsets = p.mpair == 1 ? 2 : 1;
    for (int tile = blockIdx.x; tile < total_tiles && !*abort_flag; tile += gridDim.x, ++tcount) {
      const int mg = tile / p.n_tiles, nt = tile - mg * p.n_tiles;
      const int acc = (int)(tcount % nsets);
      const uint32_t acc_ph = (tcount / nsets) & 1;
      if (!mbar_wait(&acc_full[acc], acc_ph, abort_flag)) break;
      tc_fence_after();
      const int halves = (mg * p.mpair + 1 < p.m_tiles) ? p.mpair : 1;
      for (int hf = 0; hf < halves; ++hf) {
      const int mt = mg * p.mpair + hf;
      const size_t row = (size_t)mt * kTileM + lane_grp * 32 + lane;
      size_t base = row * p.Co + (size_t)nt * p.n_tile;
      bool keep = true;
      if (p.sub == 2) {
        const size_t hw = (size_t)p.H * p.W, n = row / hw, rem = row - n * hw;
        const int h = (int)(rem / p.W), w = (int)(rem - (size_t)h * p.W);
        keep = ((h | w) & 1) == 0;
        base = (((n * (p.H >> 1) + (h >> 1)) * (p.W >> 1)) + (w >> 1)) * p.Co + (size_t)nt * p.n_tile;
      } else if (p.sub == 3) {
        const size_t hw = (size_t)p.H * p.W, n = row / hw, rem = row - n * hw;
        const int h = (int)(rem / p.W), w = (int)(rem - (size_t)h * p.W);
        base = (((n * (2 * p.H) + 2 * h) * (2 * p.W)) + 2 * w) * p.Co + (size_t)nt * p.n_tile;
      }
      const uint32_t taddr = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(acc + hf) * p.n_tile;
      for (int c0 = 0; c0 < p.n_tile; c0 += 16) {
        uint32_t v[16];
        tmem_ld16(taddr + c0, v);
        tmem_ld_wait();
        if (!keep && !stat_partial) continue;
        float f[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) f[i] = __uint_as_float(v[i]);
        if (res && keep) {
          uint4 r0 = *reinterpret_cast<const uint4*>(res + base + c0);
          uint4 r1 = *reinterpret_cast<const uint4*>(res + base + c0 + 8);
          const __nv_bfloat16* rb0 = reinterpret_cast<const __nv_bfloat16*>(&r0);
          const __nv_bfloat16* rb1 = reinterpret_cast<const __nv_bfloat16*>(&r1);
          float g[16];
#pragma unroll
          for (int i = 0; i < 8; ++i) { g[i] = __bfloat162float(rb0[i]); g[8 + i] = __bfloat162float(rb1[i]); }
          if (res_mask) {
            uint4 m0 = *reinterpret_cast<const uint4*>(res_mask + base + c0);
            uint4 m1 = *reinterpret_cast<const uint4*>(res_mask + base + c0 + 8);
            const __nv_bfloat16* mb0 = reinterpret_cast<const __nv_bfloat16*>(&m0);
            const __nv_bfloat16* mb1 = reinterpret_cast<const __nv_bfloat16*>(&m1);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              if (!(__bfloat162float(mb0[i]) > 0.f)) g[i] = 0.f;
              if (!(__bfloat162float(mb1[i]) > 0.f)) g[8 + i] = 0.f;
            }
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) f[i] += g[i];
        }
        uint4 o0, o1;
        __nv_bfloat162* ob0 = reinterpret_cast<__nv_bfloat162*>(&o0);
        __nv_bfloat162* ob1 = reinterpret_cast<__nv_bfloat162*>(&o1);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          ob0[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
          ob1[i] = __floats2bfloat162_rn(f[8 + 2 * i], f[8 + 2 * i + 1]);
        }
        if (keep) {
          *reinterpret_cast<uint4*>(out + base + c0) = o0;
          *reinterpret_cast<uint4*>(out + base + c0 + 8) = o1;
        } else {
          o0 = o1 = make_uint4(0, 0, 0, 0);
        }
        if (stat_partial) stat_add(stat_run, ew, (nt * p.n_tile + c0) >> 4, o0, o1, lane);
      }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[acc]);
    }
  }

  // Teardown.  After an abort, TMA copies may still be in flight towards this CTA's shared
  // memory: give every stage that was armed a bounded chance to complete before leaving.
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
  if (stat_partial && !*abort_flag) stat_flush(stat_run, stat_partial, p.Co);
}

// ------------------------------------------------------- patch-tile kernel ----
// Wide layers on images whose sides are multiples of 16.  conv3x3_tc_kernel fetches a 128-pixel activation tile
// again for each of the nine filter taps, and the rate at which operand rows arrive from L2 is what bounds it.
// Here a CTA works on a 16x16-pixel patch: for each 64-channel chunk ONE load brings the patch with its one-pixel
// border (18x18 pixels, out-of-bounds pixels filled with zeros: the padding) into swizzled shared memory, and
// the nine taps are nine start addresses into it.  The patch is two 128-row tiles: tile g holds pixel columns
// 8g..8g+7 of the 16 patch rows, so that consecutive 8-row groups of an operand are always one halo row (18
// pixels) apart and one shared-memory descriptor describes them.  Only the weight tiles (one per tap and chunk,
// shared by both 128-row tiles) still stream per tap.
//   A operand of (tap r,s; tile g): start = halo + ((r*18 + s + 8g) pixels), groups 18 pixels apart
//   accumulator row i of tile g  <->  patch pixel (h = i / 8, w = 8g + i % 8)
// Shared memory: two halo buffers (chunk c+1 lands while chunk c is multiplied) and a ring of weight tiles.
constexpr int kPatchThreads = 224;       // TMA warp, issuing warp of tile 0, four epilogue warps, issuing warp of tile 1
__global__ void __launch_bounds__(kPatchThreads, 1)
conv3x3_patch_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                     ConvTcParams p, __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ res,
                     const __nv_bfloat16* __restrict__ res_mask, float* __restrict__ stat_partial, int* __restrict__ error_word) {
  __shared__ float stat_run[kStatFloats];
  if (stat_partial) for (int i = threadIdx.x; i < kStatFloats; i += blockDim.x) stat_run[i] = 0.f;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* b_smem = smem + 2 * (size_t)p.halo_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(b_smem + (size_t)p.b_stages * p.b_bytes);
  uint64_t* a_full = bars;                     // [2]         TMA -> MMA, halo tiles
  uint64_t* a_empty = a_full + 2;              // [2]         MMA -> TMA
  uint64_t* full = a_empty + 2;                // [b_stages]  TMA -> MMA, weight tiles
  uint64_t* empty = full + p.b_stages;         // [b_stages]  MMA -> TMA
  uint64_t* acc_full = empty + p.b_stages;     // [3]         MMA -> epilogue, one per accumulator slot
  uint64_t* acc_empty = acc_full + 3;          // [3]         epilogue -> MMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 3);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) { mbar_init(&a_full[s], 1); mbar_init(&a_empty[s], 2); }
    for (int s = 0; s < p.b_stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 2); }
    for (int a = 0; a < 3; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(tmem_slot, p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int chunks = (p.Ci + p.kc - 1) / p.kc;
  const int pw_cnt = p.W / kPatch, ph_cnt = p.H / kPatch;
  const int total_tiles = p.N * ph_cnt * pw_cnt * p.n_tiles;
  const uint32_t halo_tx = (uint32_t)kPatchHalo * kPatchHalo * p.kc * 2;

  if (warp == 0) {
    if (lane == 0) {
      // One step = (tile, channel chunk): its halo tile, then its nine weight tiles.  The next step's halo tile is
      // requested from the middle of this step's taps: by then the multiplier has started on this step, so the
      // buffer the next tile goes to (the previous step's) has been handed back and nothing blocks here.
      uint32_t q = 0, itb = 0;                  // steps and weight tiles requested so far
      bool ok = true;
      auto load_halo = [&](int tile, int cc, uint32_t step) {
        const int pt = tile / p.n_tiles;
        const int n = pt / (ph_cnt * pw_cnt), rem = pt - n * ph_cnt * pw_cnt;
        const int ph = rem / pw_cnt, pw = rem - ph * pw_cnt;
        const int sa = step & 1;
        if (!mbar_wait(&a_empty[sa], ((step >> 1) & 1) ^ 1, abort_flag)) return false;
        mbar_expect_tx(&a_full[sa], halo_tx);
        tma_load_4d(smem + (size_t)sa * p.halo_bytes, &map_a, &a_full[sa], cc * p.kc, pw * kPatch - 1, ph * kPatch - 1, n);
        return true;
      };
      if ((int)blockIdx.x < total_tiles) ok = load_halo(blockIdx.x, 0, 0);
      for (int tile = blockIdx.x; ok && tile < total_tiles && !*abort_flag; tile += gridDim.x) {
        const int nt = tile % p.n_tiles;
        for (int cc = 0; ok && cc < chunks; ++cc, ++q) {
          // the step after this one
          int ntile = tile, ncc = cc + 1;
          if (ncc == chunks) { ncc = 0; ntile = tile + gridDim.x; }
          for (int tap = 0; tap < 9; ++tap, ++itb) {
            if (tap == 4 && ntile < total_tiles) { ok = load_halo(ntile, ncc, q + 1); if (!ok) break; }
            const int s = itb % p.b_stages;
            const uint32_t ph = (itb / p.b_stages) & 1;
            if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; break; }
            mbar_expect_tx(&full[s], p.b_tx_bytes);
            tma_load_2d(b_smem + (size_t)s * p.b_bytes, &map_b, &full[s], tap * p.Ci + cc * p.kc, nt * p.n_tile);
          }
        }
      }
    }
  } else if (warp == 1 || warp == 6) {
    // Two issuing threads, one per 128-row tile of the patch (each into its own accumulator): one thread gets a
    // tcgen05.mma out only every ~110 cycles, the pipe takes one of N = 160 every 80.
    if (lane == 0) {
      const int g = warp == 1 ? 0 : 1;
      const uint32_t idesc = instr_desc_bf16(p.n_tile);
      const uint32_t row_bytes = p.kc * 2;
      const uint32_t group_bytes = kPatchHalo * row_bytes;
      // The issuing thread is alone in its warp: every instruction it spends between two tcgen05.mma costs its full
      // latency.  All descriptors are therefore formed once, and moving an operand is a 64-bit add on the
      // descriptor's address field (16-byte units).
      uint64_t halo_desc[2], b_desc[6], tap_off[9];
      for (int i = 0; i < 2; ++i) halo_desc[i] = smem_desc_kmajor_sbo(smem_u32(smem + (size_t)i * p.halo_bytes), row_bytes, group_bytes);
      for (int i = 0; i < 6; ++i) b_desc[i] = smem_desc_kmajor(smem_u32(b_smem + (size_t)(i < p.b_stages ? i : 0) * p.b_bytes), row_bytes);
#pragma unroll
      for (int tap = 0; tap < 9; ++tap) tap_off[tap] = (uint64_t)(((tap / 3) * kPatchHalo + (tap % 3)) * row_bytes) >> 4;
      const uint64_t g_off = (uint64_t)(8 * g * row_bytes) >> 4;
      // The 128-row tiles of this CTA, numbered 2 * (patch count) + g, rotate over the accumulator slots.
      uint32_t q = 0, itb = 0, tcount = 0;
      int s = 0;
      uint32_t ph = 0;                                         // itb % b_stages and that stage's phase, kept incrementally
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles && !*abort_flag; tile += gridDim.x, ++tcount) {
        const uint32_t half = 2 * tcount + (uint32_t)g;
        const uint32_t slot = half % (uint32_t)p.acc_slots, use = half / (uint32_t)p.acc_slots;
        if (!mbar_wait(&acc_empty[slot], (use & 1) ^ 1, abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + slot * (uint32_t)p.n_tile;
        for (int cc = 0; ok && cc < chunks; ++cc, ++q) {
          const int sa = q & 1;
          if (!mbar_wait(&a_full[sa], (q >> 1) & 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          // the last chunk of a 160-channel layer holds 32 channels (the rest of its 64 is the zero fill): two K steps
          const bool short_chunk = cc == chunks - 1 && (p.Ci & 63) != 0 && (p.Ci & 63) <= 32;
#pragma unroll
          for (int tap = 0; tap < 9; ++tap, ++itb) {
            if (!mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint64_t a0 = halo_desc[sa] + tap_off[tap] + g_off, b0 = b_desc[s];
            tc_mma_bf16(d_tmem, a0, b0, idesc, (uint32_t)(cc | tap));
            tc_mma_bf16(d_tmem, a0 + 2, b0 + 2, idesc, 1);
            if (!short_chunk) {
              tc_mma_bf16(d_tmem, a0 + 4, b0 + 4, idesc, 1);
              tc_mma_bf16(d_tmem, a0 + 6, b0 + 6, idesc, 1);
            }
            tc_commit(&empty[s]);
            if (++s == p.b_stages) { s = 0; ph ^= 1; }
          }
          if (ok) tc_commit(&a_empty[sa]);
        }
        if (ok) tc_commit(&acc_full[slot]);
      }
    }
  } else if (warp >= 2 && warp <= 5) {
    const int lane_grp = warp & 3;
    uint32_t tcount = 0;
    for (int tile = blockIdx.x; tile < total_tiles && !*abort_flag; tile += gridDim.x, ++tcount) {
      const int pt = tile / p.n_tiles, nt = tile - pt * p.n_tiles;
      const int n = pt / (ph_cnt * pw_cnt), rem = pt - n * ph_cnt * pw_cnt;
      const int ph = rem / pw_cnt, pw = rem - ph * pw_cnt;
      const int i = lane_grp * 32 + lane;                       // accumulator row of this thread
      bool live = true;
      for (int g = 0; g < 2; ++g) {
        const uint32_t half = 2 * tcount + (uint32_t)g;
        const uint32_t slot = half % (uint32_t)p.acc_slots, use = half / (uint32_t)p.acc_slots;
        if (!mbar_wait(&acc_full[slot], use & 1, abort_flag)) { live = false; break; }
        tc_fence_after();
        const int h = ph * kPatch + (i >> 3), w = pw * kPatch + 8 * g + (i & 7);
        size_t base;
        bool keep = true;
        if (p.sub == 1) {
          base = (((size_t)n * p.H + h) * p.W + w) * p.Co + (size_t)nt * p.n_tile;
        } else {
          keep = ((h | w) & 1) == 0;
          base = (((size_t)n * (p.H >> 1) + (h >> 1)) * (p.W >> 1) + (w >> 1)) * p.Co + (size_t)nt * p.n_tile;
        }
        const uint32_t taddr = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + slot * (uint32_t)p.n_tile;
        for (int c0 = 0; c0 < p.n_tile; c0 += 16) {
          uint32_t v[16];
          tmem_ld16(taddr + c0, v);
          tmem_ld_wait();
          if (!keep && !stat_partial) continue;
          float f[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) f[e] = __uint_as_float(v[e]);
          if (res && keep) {
            uint4 r0 = *reinterpret_cast<const uint4*>(res + base + c0);
            uint4 r1 = *reinterpret_cast<const uint4*>(res + base + c0 + 8);
            const __nv_bfloat16* rb0 = reinterpret_cast<const __nv_bfloat16*>(&r0);
            const __nv_bfloat16* rb1 = reinterpret_cast<const __nv_bfloat16*>(&r1);
            float gq[16];
#pragma unroll
            for (int e = 0; e < 8; ++e) { gq[e] = __bfloat162float(rb0[e]); gq[8 + e] = __bfloat162float(rb1[e]); }
            if (res_mask) {
              uint4 m0 = *reinterpret_cast<const uint4*>(res_mask + base + c0);
              uint4 m1 = *reinterpret_cast<const uint4*>(res_mask + base + c0 + 8);
              const __nv_bfloat16* mb0 = reinterpret_cast<const __nv_bfloat16*>(&m0);
              const __nv_bfloat16* mb1 = reinterpret_cast<const __nv_bfloat16*>(&m1);
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
          if (keep) {
            *reinterpret_cast<uint4*>(out + base + c0) = o0;
            *reinterpret_cast<uint4*>(out + base + c0 + 8) = o1;
          } else {
            o0 = o1 = make_uint4(0, 0, 0, 0);
          }
          if (stat_partial) stat_add(stat_run, warp - 2, (nt * p.n_tile + c0) >> 4, o0, o1, lane);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[slot]);            // this tile's accumulator may be overwritten
      }
      if (!live) break;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) {
      if (error_word) atomicExch(error_word, 1);
      for (int s = 0; s < 2 + p.b_stages; ++s) {
        uint64_t* b = s < 2 ? &a_full[s] : &full[s - 2];
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
  if (stat_partial && !*abort_flag) stat_flush(stat_run, stat_partial, p.Co);
}

// ----------------------------------------------------------------- host side ---
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

inline CUtensorMapSwizzle swizzle_for(int row_bytes) {
  return row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
}

// Can this convolution run on the tensor-core kernel?  (3x3, stride 1, pad 1, channel counts
// that are multiples of 16, image rows that tile 128 pixels exactly.)
inline bool conv_tc_supported(int N, int H, int W, int Ci, int Co) {
  if (Ci % 16 || Co % 16 || Ci < 16 || Co < 16) return false;
  if (kTileM % W) return false;
  const int rows = kTileM / W;
  if (rows <= H) { if (H % rows) return false; }
  else { if (rows % H || N % (rows / H)) return false; }
  if (W > 256 || H > 256) return false;
  return true;
}

inline ConvTcParams conv_tc_params(int N, int H, int W, int Ci, int Co, int taps = 9) {
  ConvTcParams p{};
  p.W = W; p.H = H; p.N = N; p.Ci = Ci; p.Co = Co; p.sub = 1; p.taps = taps; p.act_sub = 1;
  const int rows = kTileM / W;
  if (rows <= H) { p.rows_per_tile = rows; p.imgs_per_tile = 1; }
  else { p.rows_per_tile = H; p.imgs_per_tile = rows / H; }
  // Channel chunk of a pipeline stage = one swizzle span.  Operand tiles arrive from L2 row by row, and a 128-byte
  // row costs the same as a 64-byte one, so wide layers whose channel count is not a multiple of 64 (160) still
  // take 64-channel chunks: the last chunk's surplus channels lie outside the activation tensor, are filled with
  // zeros by the hardware, and so cancel whatever weights they meet.
  p.kc = (Ci % 64 == 0 || Ci >= 128) ? 64 : (Ci % 32 == 0 ? 32 : 16);
  int nt = Co;
  if (nt > 256) { nt = 256; while (Co % nt || nt % 16) nt -= 16; }
  p.m_tiles = (int)((size_t)N * H * W / kTileM);
  // 16x16-pixel patches with their halo wherever the image allows it and the chunks are full swizzle spans
  p.patch = (taps == 9 && H % kPatch == 0 && W % kPatch == 0 && p.kc == 64) ? 1 : 0;
  // The kernel is bound by the rate at which operand tiles arrive from L2, so a weight tile is shared by two
  // 128-row tiles -- unless the layer has so few pixels (small images, many channels) that the tiles would leave
  // most SMs idle: then single 128-row tiles and narrower column tiles, down to 64, until there are about 96.
  p.mpair = p.m_tiles >= 2 ? 2 : 1;
  if (!p.patch) {
    auto tiles = [&]() { return ((p.m_tiles + p.mpair - 1) / p.mpair) * (Co / nt); };
    if (tiles() < 96) p.mpair = 1;
    while (tiles() < 96 && nt % 32 == 0 && nt / 2 >= 64 && Co % (nt / 2) == 0) nt /= 2;
  }
  p.n_tile = nt;
  p.n_tiles = Co / nt;
  p.a_bytes = (uint32_t)kTileM * p.kc * 2;
  p.b_tx_bytes = (uint32_t)nt * p.kc * 2;
  p.b_bytes = (p.b_tx_bytes + 1023u) & ~1023u;
  p.stage_bytes = (uint32_t)p.mpair * p.a_bytes + p.b_bytes;
  p.halo_bytes = ((uint32_t)kPatchHalo * kPatchHalo * p.kc * 2 + 1023u) & ~1023u;
  p.b_stages = (int)((176 * 1024 - 2 * (size_t)p.halo_bytes) / p.b_bytes);
  if (p.b_stages > 6) p.b_stages = 6;
  if (p.b_stages < 2) p.patch = 0;
  int stages = (int)(160 * 1024 / p.stage_bytes);
  p.stages = stages > 8 ? 8 : (stages < 2 ? 2 : stages);
  p.acc_slots = (p.patch && 3 * nt <= 512) ? 3 : 2;
  uint32_t cols = 32;
  while (cols < (uint32_t)(p.patch ? p.acc_slots : 2) * nt) cols <<= 1;
  p.tmem_cols = cols;
  return p;
}

inline size_t conv_tc_smem_bytes(const ConvTcParams& p) {
  if (p.patch) return 2 * (size_t)p.halo_bytes + (size_t)p.b_stages * p.b_bytes + 1024 + 256 + 64;
  return (size_t)p.stages * p.stage_bytes + 1024 + 256;
}

// act: bf16 [N][H][W][Ci]; wgt: bf16 [Co][9*Ci] (forward layout, or the flipped/transposed copy for dgrad).
inline cudaError_t conv_tc_make_maps(const ConvTcParams& p, const void* act, const void* wgt, CUtensorMap* map_a,
                                     CUtensorMap* map_b) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  const CUtensorMapSwizzle sw = swizzle_for(p.kc * 2);
  {
    // act_sub = 2: the even pixels of an [N][2H][2W][Ci] tensor are themselves a regular [N][H][W][Ci] tensor
    // with doubled pixel strides and quadrupled row and image strides
    const cuuint64_t q = (cuuint64_t)p.act_sub;
    cuuint64_t dims[4] = {(cuuint64_t)p.Ci, (cuuint64_t)p.W, (cuuint64_t)p.H, (cuuint64_t)p.N};
    cuuint64_t strides[3] = {q * p.Ci * 2, q * q * p.W * p.Ci * 2, q * q * p.H * p.W * p.Ci * 2};
    cuuint32_t box[4] = {(cuuint32_t)p.kc, (cuuint32_t)p.W, (cuuint32_t)p.rows_per_tile, (cuuint32_t)p.imgs_per_tile};
    if (p.patch) { box[1] = kPatchHalo; box[2] = kPatchHalo; box[3] = 1; }
    cuuint32_t estr[4] = {1, 1, 1, 1};
    if (enc(map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(act), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }
  {
    cuuint64_t dims[2] = {(cuuint64_t)p.taps * p.Ci, (cuuint64_t)p.Co};
    cuuint64_t strides[1] = {(cuuint64_t)p.taps * p.Ci * 2};
    cuuint32_t box[2] = {(cuuint32_t)p.kc, (cuuint32_t)p.n_tile};
    cuuint32_t estr[2] = {1, 1};
    if (enc(map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(wgt), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }
  return cudaSuccess;
}

// The kernel's dynamic shared memory exceeds the default limit: raised once (also callable up front, so
// that the first launch may happen inside a stream capture).
inline cudaError_t conv_tc_set_attrs() {
  static bool attr_set = false;
  if (attr_set) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(conv3x3_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(conv3x3_patch_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e == cudaSuccess) attr_set = true;
  return e;
}

// `stat_partial` (nullable): room for one row of 2 * Co floats per CTA (at most sm_count rows); *ctas_out = rows written.
inline cudaError_t conv_tc_launch(cudaStream_t st, const ConvTcParams& p, const CUtensorMap& map_a,
                                  const CUtensorMap& map_b, __nv_bfloat16* out, const __nv_bfloat16* res,
                                  const __nv_bfloat16* res_mask, int* error_word, int sm_count,
                                  float* stat_partial = nullptr, int* ctas_out = nullptr) {
  const size_t smem = conv_tc_smem_bytes(p);
  {
    cudaError_t e = conv_tc_set_attrs();
    if (e != cudaSuccess) return e;
  }
  if (p.patch) {
    const int tiles = p.N * (p.H / kPatch) * (p.W / kPatch) * p.n_tiles;
    const int grid = tiles < sm_count ? tiles : sm_count;
    if (ctas_out) *ctas_out = grid;
    conv3x3_patch_kernel<<<grid, kPatchThreads, smem, st>>>(map_a, map_b, p, out, res, res_mask, stat_partial, error_word);
    return cudaGetLastError();
  }
  const int tiles = ((p.m_tiles + p.mpair - 1) / p.mpair) * p.n_tiles;
  const int grid = tiles < sm_count ? tiles : sm_count;
  if (ctas_out) *ctas_out = grid;
  conv3x3_tc_kernel<<<grid, kThreads, smem, st>>>(map_a, map_b, p, out, res, res_mask, stat_partial, error_word);
  return cudaGetLastError();
}

// Probe of the tensor pipe's instruction rate, for the roofline arguments about the kernels above: one thread of one
// CTA per SM issues `reps` x 4 x `accs` instructions (M = 128, N = n, K = 16, bf16, both operands K-major in
// 128-byte-swizzled shared memory whose contents do not matter) back to back, rotating over `accs` accumulators, and
// waits for the last one.  out[0] = cycles until the last one was issued, out[1] = until it completed (CTA 0).
// `unrolled` = 0 keeps the rotation over the accumulators as a run-time loop: the same instructions with a loop
// counter and a branch between them, which is what an issuing loop that is not unrolled looks like.
__global__ void __launch_bounds__(128, 1) mma_rate_kernel(int n, int accs, int reps, int unrolled, long long* __restrict__ out,
                                                          int* __restrict__ error_word) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t slot;
  __shared__ int flag;
  volatile int* abort_flag = &flag;
  // A: 128 rows x 128 bytes; B: 256 rows x 128 bytes; finite values
  for (int i = threadIdx.x; i < 48 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0x3c003c00u;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (threadIdx.x < 32) tmem_alloc(&slot, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = slot;
  if (threadIdx.x == 0) {
    const uint32_t a_addr = smem_u32(smem), b_addr = a_addr + 16 * 1024;
    const uint64_t a = smem_desc_kmajor(a_addr, 128), b = smem_desc_kmajor(b_addr, 128);
    const uint32_t idesc = instr_desc_bf16(n);
    const long long t0 = clock64();
    const uint32_t d1 = tmem + (uint32_t)n, d2 = tmem + 2u * (uint32_t)n;
    if (unrolled) {
      for (int r = 0; r < reps; ++r) {
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          tc_mma_bf16(tmem, a + 2 * ks, b + 2 * ks, idesc, 1);
          if (accs >= 2) tc_mma_bf16(d1, a + 2 * ks, b + 2 * ks, idesc, 1);
          if (accs >= 3) tc_mma_bf16(d2, a + 2 * ks, b + 2 * ks, idesc, 1);
        }
      }
    } else {
      for (int r = 0; r < reps; ++r)
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll 1
          for (int q = 0; q < accs; ++q) tc_mma_bf16(tmem + (uint32_t)(q * n), a + 2 * ks, b + 2 * ks, idesc, 1);
    }
    const long long t1 = clock64();
    tc_commit(&bar);
    mbar_wait(&bar, 0, abort_flag);
    const long long t2 = clock64();
    if (blockIdx.x == 0) { out[0] = t1 - t0; out[1] = t2 - t0; }
    if (*abort_flag && error_word) atomicExch(error_word, 1);
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// Flipped / transposed weight copy for the data gradient of a 3x3 convolution (taps = 9):
// dst[ci][2-r][2-s][co] = src[co][r][s][ci]; taps = 1: the transpose of a 1x1 filter.  One block row per entry of
// `table` (src offset, dst offset, Co, Ci, taps), all offsets in elements from the two base pointers.
struct FlipEntry { unsigned long long src, dst; int Co, Ci, taps; };
// The copy of one entry by the blocks blockIdx.x = 0 .. gridDim.x-1 (256 threads each).  Tiles of one tap's [Co][Ci]
// matrix go through shared memory, so that both the reads (along ci) and the writes (along co) are contiguous.
__device__ __forceinline__ void wflip_entry(const __nv_bfloat16* __restrict__ src_base, __nv_bfloat16* __restrict__ dst_base,
                                            const FlipEntry& e, __nv_bfloat16 (&tile)[64][66]) {
  const int T = e.taps;                                                       // 9, or 1: the plain transpose of a 1x1 filter
  if (((e.Co | e.Ci) & 7) == 0 &&
      ((reinterpret_cast<uintptr_t>(src_base + e.src) | reinterpret_cast<uintptr_t>(dst_base + e.dst)) & 15) == 0) {
    // 64 x 64 tiles moved as 16-byte vectors (8 channels): a thread reads two vectors along ci, then writes two along co
    // that it gathers from eight rows of the tile.  Rows are 66 elements = 33 words apart: the word-wise stores of a
    // warp (4 rows x 8 vectors) fall on 32 different banks, the gathers (rows 8 apart) meet two by two.
    const int tco = (e.Co + 63) / 64, tci = (e.Ci + 63) / 64;
    const int total = T * tco * tci;
    const int vr = threadIdx.x >> 3, vc = (threadIdx.x & 7) * 8;                // vector slot: row 0..31 (+32), column 0,8,..56
    for (int id = blockIdx.x; id < total; id += gridDim.x) {
      const int t = id / (tco * tci), rem = id - t * tco * tci;
      const int co0 = (rem / tci) * 64, ci0 = (rem - (rem / tci) * tci) * 64;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int co = co0 + vr + 32 * h, ci = ci0 + vc;
        if (co < e.Co && ci < e.Ci) {
          const uint4 v = *reinterpret_cast<const uint4*>(src_base + e.src + ((size_t)co * T + t) * e.Ci + ci);
          uint32_t* d = reinterpret_cast<uint32_t*>(&tile[vr + 32 * h][vc]);
          d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
        }
      }
      __syncthreads();
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int ci = ci0 + vr + 32 * h, co = co0 + vc;
        if (co < e.Co && ci < e.Ci) {
          uint4 v;
          __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(&v);
#pragma unroll
          for (int j = 0; j < 8; ++j) o[j] = tile[vc + j][vr + 32 * h];
          *reinterpret_cast<uint4*>(dst_base + e.dst + ((size_t)ci * T + (T - 1 - t)) * e.Co + co) = v;
        }
      }
      __syncthreads();
    }
    return;
  }
  // any channel counts and offsets: 32 x 32 tiles, element by element; 256 threads = 32 columns x 8 rows
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int tco = (e.Co + 31) / 32, tci = (e.Ci + 31) / 32;
  const int total = T * tco * tci;
  for (int id = blockIdx.x; id < total; id += gridDim.x) {
    const int t = id / (tco * tci), rem = id - t * tco * tci;
    const int co0 = (rem / tci) * 32, ci0 = (rem - (rem / tci) * tci) * 32;
    for (int j = ty; j < 32; j += 8) {
      const int co = co0 + j, ci = ci0 + tx;
      if (co < e.Co && ci < e.Ci) tile[j][tx] = src_base[e.src + ((size_t)co * T + t) * e.Ci + ci];
    }
    __syncthreads();
    for (int j = ty; j < 32; j += 8) {
      const int ci = ci0 + j, co = co0 + tx;
      if (co < e.Co && ci < e.Ci) dst_base[e.dst + ((size_t)ci * T + (T - 1 - t)) * e.Co + co] = tile[tx][j];
    }
    __syncthreads();
  }
}
__global__ void __launch_bounds__(256) wflip_kernel(const __nv_bfloat16* __restrict__ src_base, __nv_bfloat16* __restrict__ dst_base,
                                                    const FlipEntry* __restrict__ table) {
  __shared__ __align__(16) __nv_bfloat16 tile[64][66];
  wflip_entry(src_base, dst_base, table[blockIdx.y], tile);
}
// One filter, its entry passed by value.
__global__ void __launch_bounds__(256) wflip_one_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, FlipEntry e) {
  __shared__ __align__(16) __nv_bfloat16 tile[64][66];
  wflip_entry(src, dst, e, tile);
}

}  // namespace tc
}  // namespace fdg
