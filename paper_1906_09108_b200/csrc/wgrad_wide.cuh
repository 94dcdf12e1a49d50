// Weight gradient of 3x3 / stride 1 / pad 1 convolutions of WIDE layers (128 channels and more), and of 1x1
// convolutions (projection shortcuts, 64 channels and more), on the sm_100a tensor cores, on exact pixel tiles:
//
//   dW[co][r][s][ci] = sum over pixels (n,h,w) of dY[n][h][w][co] * X[n][h+r-1][w+s-1][ci]          (3x3)
//   dW[co][ci]       = sum over pixels (n,h,w) of dY[n][h][w][co] * X[n][h][w][ci]                  (1x1)
//
// Pixels are the reduction dimension, so both operands are read MN-major (channels contiguous).  A CTA
// owns one output tile -- 128 output channels x one filter row r x its taps s x up to 160 input
// channels: one fp32 accumulator of 128 x nci per tap in tensor memory (<= 480 of its 512 columns) -- and a
// share of the pixels, which it walks in SLABS of 64 pixels (S = 64/W image rows of one image):
//   dY slab: [S*W pixels][128 co]     as two 64-channel sub-tiles, one 128-byte swizzle span per pixel
//   X  slab: 3x3: [S*(W+2) pixels][nci ci], rows h0+r-1 .. h0+r-2+S with the border columns -1 and W (out-of-
//            bounds rows and columns are the hardware's zero fill = the padding); 1x1: [S*W pixels][nci ci];
//            64-channel sub-tiles either way
// One instruction takes 16 pixels: 16 consecutive pixels of an image row (W >= 16) or two rows of 8
// (W = 8: the second 8-pixel group of the X slab lies one slab row further on, which is the descriptor's
// stride between 8-row groups).  For tap s the X operand simply starts s pixels later, so the dY block
// is read once for three instructions and no multiplication is spent on border pixels.
// The CTAs that share an output tile write their partial sums to scratch; a second kernel adds them in
// CTA order, so the result does not depend on scheduling.
//
// Roles by warp: 0 = TMA producer, 1 = MMA issuer (one elected lane), 2..5 = write-out (32 tensor-memory
// lanes each).  Every wait is bounded; on time-out the CTA raises an error word.
#pragma once
#include "conv_halo.cuh"

namespace fdg {
namespace wide {

using namespace fdg::tc;

constexpr int kWideThreads = 192;
constexpr int kSlabPixels = 64;
constexpr int kCoBlock = 128;
constexpr size_t kWideSmemBudget = 200 * 1024;

struct WideParams {
  int N, H, W, Wp;
  int Ci, Co;
  int nci;                  // input channels per CTA = N of the instruction (multiple of 16, <= 160)
  int ci_chunks, co_blocks;
  int xsub;                 // 64-channel sub-tiles of the X slab: ceil(nci / 64)
  int taps;                 // 3: one filter row of a 3x3 filter (pad 1); 1: a 1x1 filter (no padding)
  int rdim;                 // filter rows: 3 or 1 (the CTAs of blockIdx.x % rdim share everything but r)
  int xw;                   // pixels per image row of the X slab: W + 2 with the border columns, W without
  int S;                    // image rows per slab
  int slabs;                // N * H / S
  int splits;               // CTAs per output tile
  int stages;
  uint32_t y_sub_bytes, x_sub_bytes;      // one 64-channel sub-tile of each slab (multiples of 1 KiB)
  uint32_t y_bytes, x_bytes;              // per stage
  uint32_t tx_bytes;                      // what TMA moves per stage
  uint32_t sbo_x;                         // bytes between the two 8-pixel groups of an instruction in the X slab
  uint32_t tmem_cols;
};

// Shared-memory descriptor of an MN-major operand in 128-byte-swizzled rows (one k per row, 64 channels wide):
// `lbo` = bytes between consecutive 64-channel blocks, `sbo` = bytes between consecutive 8-row k groups.
__device__ __forceinline__ uint64_t desc_mn128(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

template <int TAPS>
__global__ void __launch_bounds__(kWideThreads, 1)
wgrad_wide_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y, WideParams p,
                  float* __restrict__ partial, int* __restrict__ error_word) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t stage_bytes = p.y_bytes + p.x_bytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)p.stages * stage_bytes);
  uint64_t* empty = full + p.stages;
  uint64_t* done = empty + p.stages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(done + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // output tile of this CTA: blockIdx.x = (co block * ci chunks + ci chunk) * rdim + r
  const int r = (int)blockIdx.x % p.rdim;
  const int pair = (int)blockIdx.x / p.rdim;
  const int chunk = pair % p.ci_chunks, cob = pair / p.ci_chunks;
  const int ci0 = chunk * p.nci, co0 = cob * kCoBlock;
  const int slabs_per_img = p.H / p.S;

  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_x)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_y)) : "memory");
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(done, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(tmem_slot, p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      for (int slab = blockIdx.y; slab < p.slabs && !*abort_flag; slab += gridDim.y, ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) break;
        const int n = slab / slabs_per_img, h0 = (slab - n * slabs_per_img) * p.S;
        uint8_t* ys = smem + (size_t)s * stage_bytes;
        uint8_t* xs = ys + p.y_bytes;
        mbar_expect_tx(&full[s], p.tx_bytes);
        for (int j = 0; j < 2; ++j) tma_load_4d(ys + (size_t)j * p.y_sub_bytes, &map_y, &full[s], co0 + 64 * j, 0, h0, n);
        for (int j = 0; j < p.xsub; ++j)
          tma_load_4d(xs + (size_t)j * p.x_sub_bytes, &map_x, &full[s], ci0 + 64 * j, p.taps == 3 ? -1 : 0,
                      p.taps == 3 ? h0 + r - 1 : h0, n);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // The issuing thread is alone in its warp, so every instruction between two tcgen05.mma costs its full
      // latency: the descriptors of a stage are formed once, a reduction step moves them by additions on the
      // address field (16-byte units), and the loops over steps and taps are unrolled.
      const uint32_t idesc = halo::instr_desc(p.nci, true);
      constexpr int ksteps = kSlabPixels / 16;
      const uint32_t y_first = smem_u32(smem);
      const uint64_t a_first = desc_mn128(y_first, p.y_sub_bytes, 1024u);
      const uint64_t b_first = desc_mn128(y_first + p.y_bytes, p.x_sub_bytes, p.sbo_x);
      const uint64_t stage_units = (uint64_t)(stage_bytes >> 4);
      uint64_t b_off[ksteps];
      for (int ks = 0; ks < ksteps; ++ks) {
        const int pix = ks * 16;                                 // first pixel of the step inside the dY slab
        const int row = pix / p.W, col = pix - row * p.W;        // W = 8: row is even and the step takes rows row, row+1
        b_off[ks] = (uint64_t)((row * p.xw + col) * 8);          // one pixel = 128 bytes = 8 units
      }
      const uint32_t d1 = tmem_base + (uint32_t)p.nci, d2 = tmem_base + 2u * (uint32_t)p.nci;
      uint32_t it = 0;
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int slab = blockIdx.y; slab < p.slabs && !*abort_flag; slab += gridDim.y, ++it) {
        if (!mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint64_t a0 = a_first + (uint64_t)s * stage_units, b0 = b_first + (uint64_t)s * stage_units;
#pragma unroll
        for (int ks = 0; ks < ksteps; ++ks) {
          const uint64_t a = a0 + (uint64_t)(ks * 128), b = b0 + b_off[ks];      // 16 pixels = 2048 bytes = 128 units
          const uint32_t acc = (it | (uint32_t)ks) != 0;
          tc_mma_bf16(tmem_base, a, b, idesc, acc);
          if (TAPS == 3) {
            tc_mma_bf16(d1, a, b + 8, idesc, acc);
            tc_mma_bf16(d2, a, b + 16, idesc, acc);
          }
        }
        tc_commit(&empty[s]);
        if (++s == p.stages) { s = 0; ph ^= 1; }
      }
      if (ok) tc_commit(done);
    }
  } else {
    // Write-out.  A lane holds one output row (an output channel) of the accumulators; written straight from
    // registers, a warp's store would touch 32 rows 11 KB apart with 16 bytes each.  Each 32 x 32 block therefore
    // goes through shared memory (the pipeline's stages are idle by now) and leaves as 128-byte row segments.
    const int lane_grp = warp & 3;
    if (mbar_wait(done, 0, abort_flag)) {
      tc_fence_after();
      float* stage = reinterpret_cast<float*>(smem) + (size_t)lane_grp * (32 * 33);   // this warp's [32][33] block
      const int row_base = co0 + lane_grp * 32;
      const size_t ftaps = (size_t)p.rdim * p.taps;                        // taps of the whole filter: 9 or 1
      const size_t row_stride = ftaps * p.Ci;
      float* dst = partial + (size_t)blockIdx.y * ((size_t)p.Co * row_stride) + ((size_t)row_base * ftaps + (size_t)r * p.taps) * p.Ci + ci0;
      const int sub_row = lane >> 3, col4 = (lane & 7) * 4;                // write-out: 4 rows x 8 lanes x 4 columns
      for (int sx = 0; sx < p.taps; ++sx) {
        for (int c0 = 0; c0 < p.nci; c0 += 32) {
          const int ncol = min(32, p.nci - c0);                            // 32, or 16 at the end of a chunk
          uint32_t v[16];
          tmem_ld16(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(sx * p.nci + c0), v);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 16; ++e) stage[lane * 33 + e] = __uint_as_float(v[e]);
          if (ncol == 32) {
            tmem_ld16(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(sx * p.nci + c0 + 16), v);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 16; ++e) stage[lane * 33 + 16 + e] = __uint_as_float(v[e]);
          }
          __syncwarp();
          if (col4 < ncol && ci0 + c0 + col4 < p.Ci) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int rr = i * 4 + sub_row;
              if (row_base + rr < p.Co) {
                const float* src = stage + rr * 33 + col4;
                *reinterpret_cast<float4*>(dst + (size_t)rr * row_stride + (size_t)sx * p.Ci + c0 + col4) =
                    make_float4(src[0], src[1], src[2], src[3]);
              }
            }
          }
          __syncwarp();
        }
      }
    }
  }

  // Teardown.  After an abort, TMA copies may still be in flight towards this CTA's shared memory:
  // give every stage that was armed a bounded chance to complete before leaving.
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

// dw[i] = partial[0][i] + partial[1][i] + ... in split order; four consecutive outputs per thread.
__global__ void __launch_bounds__(256) wgrad_wide_sum_kernel(const float4* __restrict__ partial, float4* __restrict__ dw,
                                                             size_t n4, int splits) {
  grid_dependency_wait();                 // launched ahead of the end of the kernel that writes `partial`
  const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= n4) return;
  float4 a = partial[i];
  for (int j = 1; j < splits; ++j) {
    const float4 b = partial[(size_t)j * n4 + i];
    a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
  }
  dw[i] = a;
}

// ----------------------------------------------------------------- host side ---
inline int wide_nci(int Ci) {
  if (Ci % 160 == 0) return 160;
  if (Ci % 128 == 0) return 128;
  if (Ci <= 160) return Ci;
  return 0;
}

// R = 3: x and dy are [N][H][W][.]; R = 1: dy is [N][H][W][Co] and x the tensor of the same pixels (for stride 2, the
// even pixels of the layer input, see make_slab_map).
inline WideParams wide_params(int N, int H, int W, int Ci, int Co, int sm_count, int R = 3) {
  WideParams p{};
  p.N = N; p.H = H; p.W = W; p.Wp = W + 2; p.Ci = Ci; p.Co = Co;
  p.taps = R; p.rdim = R; p.xw = R == 3 ? W + 2 : W;
  p.nci = wide_nci(Ci);
  if (p.nci == 0 || W < 8 || kSlabPixels % W) { p.stages = 0; return p; }
  p.S = kSlabPixels / W;
  if (H % p.S) { p.stages = 0; return p; }
  p.ci_chunks = Ci / p.nci;
  p.co_blocks = (Co + kCoBlock - 1) / kCoBlock;
  p.xsub = (p.nci + 63) / 64;
  p.slabs = N * (H / p.S);
  p.y_sub_bytes = kSlabPixels * 128;
  p.x_sub_bytes = halo::round_up_u32((uint32_t)(p.S * p.xw) * 128u, 1024);
  p.y_bytes = 2 * p.y_sub_bytes;
  p.x_bytes = (uint32_t)p.xsub * p.x_sub_bytes;
  p.tx_bytes = 2 * p.y_sub_bytes + (uint32_t)p.xsub * (uint32_t)(p.S * p.xw) * 128u;
  p.sbo_x = W == 8 ? (uint32_t)p.xw * 128u : 1024u;
  int stages = (int)((kWideSmemBudget - 2048) / (p.y_bytes + p.x_bytes));
  if (stages > 6) stages = 6;
  p.stages = stages;
  uint32_t cols = 32;
  while (cols < (uint32_t)(p.taps * p.nci)) cols <<= 1;
  p.tmem_cols = cols;
  const int tiles = p.co_blocks * p.ci_chunks * p.rdim;
  const int sms = sm_count > 0 ? sm_count : 148;
  int splits = sms / tiles;
  if (splits < 1) splits = 1;
  if (splits > 32) splits = 32;
  if (splits > p.slabs) splits = p.slabs;
  p.splits = splits;
  return p;
}
inline size_t wide_smem_bytes(const WideParams& p) {
  return (size_t)p.stages * ((size_t)p.y_bytes + p.x_bytes) + (size_t)(2 * p.stages + 1) * 8 + 16 + 1024;
}
// 64 channels and more on both sides (a 64-channel sub-tile is one swizzle span).  Narrow 3x3 layers that the
// halo-tile kernel covers are left to it by the dispatcher: they are bound by memory traffic, where its single
// pass over whole images wins.
inline bool wide_supported(int N, int H, int W, int Ci, int Co, int R = 3) {
  if (Ci < 64 || Co < 64 || Ci % 16 || Co % 16 || N < 1 || H < 1) return false;
  WideParams p = wide_params(N, H, W, Ci, Co, 148, R);
  return p.stages >= 2 && p.tmem_cols <= 512 && p.co_blocks * p.ci_chunks * p.rdim <= 65535;
}
// fp32 elements of scratch for the per-split partial sums (sized for a 148-SM split).
inline size_t wide_scratch_elems(int N, int H, int W, int Ci, int Co, int R = 3) {
  WideParams p = wide_params(N, H, W, Ci, Co, 148, R);
  return (size_t)p.splits * Co * R * R * Ci;
}

// bf16 NHWC tensor map with a box of 64 channels x box_w pixels x box_h rows of one image, 128-byte swizzle.
// sub = 2: `act` is an [N][2H][2W][C] tensor of which only the even pixels are addressed (they form a regular
// [N][H][W][C] tensor with doubled pixel and quadrupled row strides).
inline cudaError_t make_slab_map(const void* act, int N, int H, int W, int C, int box_w, int box_h, CUtensorMap* map, int sub = 1) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  const cuuint64_t q = (cuuint64_t)sub;
  cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
  cuuint64_t strides[3] = {q * C * 2, q * q * W * C * 2, q * q * H * W * C * 2};
  cuuint32_t box[4] = {64u, (cuuint32_t)box_w, (cuuint32_t)box_h, 1u};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  if (enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(act), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  return cudaSuccess;
}

inline cudaError_t wide_set_attrs() {
  static bool done = false;
  if (done) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(wgrad_wide_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWideSmemBudget + 8192);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(wgrad_wide_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWideSmemBudget + 8192);
  if (e == cudaSuccess) done = true;
  return e;
}

}  // namespace wide
}  // namespace fdg
