// Convolution forward, data gradient and weight gradient on the CUDA cores, fp32
// accumulation: the exact-arithmetic mode of the library and the fallback for
// shapes the tensor-core kernels do not take (3-channel stem, strided and 1x1
// convolutions, channel counts that are not multiples of 16).
//
// All three are one tiled GEMM  C[m][n] = sum_k A(m,k) * B(k,n)  whose operands are
// gathered on the fly (implicit GEMM, nothing is materialised):
//   FPROP  m = output pixel (n,p,q)  n = c_out        k = (r,s,c_in)
//          A = x[n, p*st+r-pad, q*st+s-pad, c_in]     B = w[c_out][r][s][c_in]
//   DGRAD  m = input pixel (n,h,w)   n = c_in         k = (r,s,c_out)
//          A = dy[n, (h+pad-r)/st, (w+pad-s)/st, c_out] where divisible and in range
//          B = w[c_out][r][s][c_in]
//   FPROP and DGRAD may add a residual tensor (optionally gated by [mask > 0]) to C.
//   WGRAD  m = (r,s,c_in)            n = c_out        k = output pixel, split over gridDim.z
//          A = x[n, p*st+r-pad, q*st+s-pad, c_in]     B = dy[pixel][c_out]
//          C -> partial[z][c_out][r][s][c_in], summed over z in a fixed order afterwards
#pragma once
#include <algorithm>
#include <type_traits>

#include "elementwise.cuh"

namespace fdg {

struct ConvGeom {
  int N, H, W, Ci;      // input  tensor [N][H][W][Ci]
  int P, Q, Co;         // output tensor [N][P][Q][Co]
  int R, S, stride, pad;
};

enum { CONV_FPROP = 0, CONV_DGRAD = 1, CONV_WGRAD = 2 };
constexpr int kSimtBK = 16;
constexpr int kSimtThreads = 256;

template <typename T, int MODE, int BM, int BN, int TM, int TN>
__global__ void __launch_bounds__(kSimtThreads)
conv_simt_kernel(ConvGeom g, const T* __restrict__ act,      // FPROP/WGRAD: x ; DGRAD: dy
                 const T* __restrict__ wgt,                  // FPROP/DGRAD: w ; WGRAD: dy
                 T* __restrict__ out,                        // FPROP: y ; DGRAD: dx ; WGRAD: unused
                 float* __restrict__ wpartial,               // WGRAD: [gridDim.z][Co*R*S*Ci]
                 const T* __restrict__ res,                  // FPROP/DGRAD: optional addend, same shape as the output
                 const T* __restrict__ res_mask,             // optional: the addend counts only where mask > 0
                 int k_chunk) {                              // WGRAD: pixels per z-slice (multiple of BK)
  static_assert((BM / TM) * (BN / TN) == kSimtThreads, "tile/thread mismatch");
  constexpr int BK = kSimtBK;
  __shared__ float As[BK][BM + 1];
  __shared__ float Bs[BK][BN + 1];

  const int tid = threadIdx.x;
  const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
  int Mdim, Ndim, Kdim;
  if (MODE == CONV_FPROP) { Mdim = g.N * g.P * g.Q; Ndim = g.Co; Kdim = g.R * g.S * g.Ci; }
  else if (MODE == CONV_DGRAD) { Mdim = g.N * g.H * g.W; Ndim = g.Ci; Kdim = g.R * g.S * g.Co; }
  else { Mdim = g.R * g.S * g.Ci; Ndim = g.Co; Kdim = g.N * g.P * g.Q; }
  int kbeg = 0, kend = Kdim;
  if (MODE == CONV_WGRAD) { kbeg = blockIdx.z * k_chunk; kend = min(kbeg + k_chunk, Kdim); }

  const int tx = tid % (BN / TN), ty = tid / (BN / TN);
  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  // ---- loader geometry -------------------------------------------------------
  // FPROP/DGRAD: A is contiguous along k -> thread owns column kk = tid%BK and rows tid/BK + j*16.
  // WGRAD:       A is contiguous along m -> thread owns row   mm = tid%BM and columns tid/BM + j*(256/BM).
  constexpr int A_PER = BM * BK / kSimtThreads;
  constexpr int B_PER = (BN * BK + kSimtThreads - 1) / kSimtThreads;
  int a_n[A_PER], a_h[A_PER], a_w[A_PER];       // decoded pixel of each owned row (FPROP/DGRAD)
  if (MODE != CONV_WGRAD) {
#pragma unroll
    for (int j = 0; j < A_PER; ++j) {
      int m = m0 + tid / BK + j * (kSimtThreads / BK);
      if (m < Mdim) {
        int hw = (MODE == CONV_FPROP) ? g.P * g.Q : g.H * g.W;
        int wd = (MODE == CONV_FPROP) ? g.Q : g.W;
        int n = m / hw, rem = m - n * hw;
        a_n[j] = n; a_h[j] = rem / wd; a_w[j] = rem - a_h[j] * wd;
      } else {
        a_n[j] = -1; a_h[j] = 0; a_w[j] = 0;
      }
    }
  }
  int wm_r = 0, wm_s = 0, wm_c = 0;             // decoded (r,s,ci) of the owned row (WGRAD)
  bool wm_ok = false;
  if (MODE == CONV_WGRAD) {
    int m = m0 + tid % BM;
    wm_ok = m < Mdim;
    if (wm_ok) { wm_r = m / (g.S * g.Ci); int rem = m - wm_r * g.S * g.Ci; wm_s = rem / g.Ci; wm_c = rem - wm_s * g.Ci; }
  }

  for (int k0 = kbeg; k0 < kend; k0 += BK) {
    // ---- A tile ---------------------------------------------------------------
    if (MODE == CONV_FPROP) {
      const int kk = tid % BK, k = k0 + kk;
      int r = 0, s = 0, c = 0;
      const bool kok = k < kend;
      if (kok) { r = k / (g.S * g.Ci); int rem = k - r * g.S * g.Ci; s = rem / g.Ci; c = rem - s * g.Ci; }
#pragma unroll
      for (int j = 0; j < A_PER; ++j) {
        float v = 0.f;
        if (kok && a_n[j] >= 0) {
          int h = a_h[j] * g.stride + r - g.pad, w = a_w[j] * g.stride + s - g.pad;
          if (h >= 0 && h < g.H && w >= 0 && w < g.W)
            v = to_f(act[(((size_t)a_n[j] * g.H + h) * g.W + w) * g.Ci + c]);
        }
        As[kk][tid / BK + j * (kSimtThreads / BK)] = v;
      }
    } else if (MODE == CONV_DGRAD) {
      const int kk = tid % BK, k = k0 + kk;
      int r = 0, s = 0, c = 0;
      const bool kok = k < kend;
      if (kok) { r = k / (g.S * g.Co); int rem = k - r * g.S * g.Co; s = rem / g.Co; c = rem - s * g.Co; }
#pragma unroll
      for (int j = 0; j < A_PER; ++j) {
        float v = 0.f;
        if (kok && a_n[j] >= 0) {
          int hp = a_h[j] + g.pad - r, wq = a_w[j] + g.pad - s;
          if (hp >= 0 && wq >= 0 && hp % g.stride == 0 && wq % g.stride == 0) {
            int p = hp / g.stride, q = wq / g.stride;
            if (p < g.P && q < g.Q) v = to_f(act[(((size_t)a_n[j] * g.P + p) * g.Q + q) * g.Co + c]);
          }
        }
        As[kk][tid / BK + j * (kSimtThreads / BK)] = v;
      }
    } else {
      const int mm = tid % BM;
#pragma unroll
      for (int j = 0; j < A_PER; ++j) {
        const int kk = tid / BM + j * (kSimtThreads / BM);
        const int k = k0 + kk;
        float v = 0.f;
        if (wm_ok && k < kend) {
          int n = k / (g.P * g.Q), rem = k - n * g.P * g.Q;
          int p = rem / g.Q, q = rem - p * g.Q;
          int h = p * g.stride + wm_r - g.pad, w = q * g.stride + wm_s - g.pad;
          if (h >= 0 && h < g.H && w >= 0 && w < g.W) v = to_f(act[(((size_t)n * g.H + h) * g.W + w) * g.Ci + wm_c]);
        }
        As[kk][mm] = v;
      }
    }
    // ---- B tile ---------------------------------------------------------------
#pragma unroll
    for (int j = 0; j < B_PER; ++j) {
      const int e = tid + j * kSimtThreads;
      if (e < BN * BK) {
        float v = 0.f;
        if (MODE == CONV_FPROP) {
          const int kk = e % BK, nn = e / BK;
          const int k = k0 + kk, n = n0 + nn;
          if (k < kend && n < Ndim) v = to_f(wgt[(size_t)n * Kdim + k]);
          Bs[kk][nn] = v;
        } else if (MODE == CONV_DGRAD) {
          const int nn = e % BN, kk = e / BN;
          const int k = k0 + kk, n = n0 + nn;
          if (k < kend && n < Ndim) {
            int r = k / (g.S * g.Co), rem = k - r * g.S * g.Co;
            int s = rem / g.Co, co = rem - s * g.Co;
            v = to_f(wgt[(((size_t)co * g.R + r) * g.S + s) * g.Ci + n]);
          }
          Bs[kk][nn] = v;
        } else {
          const int nn = e % BN, kk = e / BN;
          const int k = k0 + kk, n = n0 + nn;
          if (k < kend && n < Ndim) v = to_f(wgt[(size_t)k * g.Co + n]);
          Bs[kk][nn] = v;
        }
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[TM], b[TN];
#pragma unroll
      for (int i = 0; i < TM; ++i) a[i] = As[kk][ty * TM + i];
#pragma unroll
      for (int j = 0; j < TN; ++j) b[j] = Bs[kk][tx * TN + j];
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

  // ---- epilogue ---------------------------------------------------------------
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int m = m0 + ty * TM + i;
    if (m >= Mdim) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int n = n0 + tx * TN + j;
      if (n >= Ndim) continue;
      if (MODE == CONV_WGRAD) {
        wpartial[(size_t)blockIdx.z * Mdim * Ndim + (size_t)n * Mdim + m] = acc[i][j];
      } else {
        const size_t idx = (size_t)m * Ndim + n;
        float v = acc[i][j];
        if (res) {
          float r = to_f(res[idx]);
          if (res_mask && !(to_f(res_mask[idx]) > 0.f)) r = 0.f;
          v += r;
        }
        out[idx] = from_f<T>(v);
      }
    }
  }
}

// grad[i] = sum_z partial[z][i], z ascending.
__global__ void wgrad_reduce_kernel(const float* __restrict__ partial, float* __restrict__ grad, size_t n, int splits) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    float a = 0.f;
    for (int z = 0; z < splits; ++z) a += partial[(size_t)z * n + i];
    grad[i] = a;
  }
}

// The same sum for many partial rows of a short vector (one row per image): a block takes 32 consecutive outputs,
// its 16 warps every 16th row (a warp reads 128 contiguous bytes of a row), and the 16 partial sums of an output are
// added in warp order, so the result does not depend on scheduling.
__global__ void __launch_bounds__(512) wgrad_reduce_tall_kernel(const float* __restrict__ partial, float* __restrict__ grad,
                                                                size_t n, int splits) {
  __shared__ float part[16][33];
  const int col = threadIdx.x & 31, rg = threadIdx.x >> 5;
  const size_t i = (size_t)blockIdx.x * 32 + col;
  float a = 0.f;
  if (i < n) {
#pragma unroll 4
    for (int z = rg; z < splits; z += 16) a += partial[(size_t)z * n + i];
  }
  part[rg][col] = a;
  __syncthreads();
  if (rg == 0 && i < n) {
    float t = 0.f;
#pragma unroll
    for (int r = 0; r < 16; ++r) t += part[r][col];
    grad[i] = t;
  }
}
// grad = the sum of `splits` partial rows of n floats, on stream st.
inline cudaError_t launch_wgrad_reduce(cudaStream_t st, const float* partial, float* grad, size_t n, int splits) {
  if (splits >= 32 && n <= (size_t)1 << 16) {
    wgrad_reduce_tall_kernel<<<(unsigned)((n + 31) / 32), 512, 0, st>>>(partial, grad, n, splits);
  } else {
    int blocks = (int)((n + 255) / 256); if (blocks > 1184) blocks = 1184;
    wgrad_reduce_kernel<<<blocks, 256, 0, st>>>(partial, grad, n, splits);
  }
  return cudaGetLastError();
}

// Number of pixel slices the weight-gradient GEMM is split into, and the slice length.
inline void wgrad_split(const ConvGeom& g, int bm, int bn, int* splits, int* k_chunk) {
  const long M = (long)g.R * g.S * g.Ci, N = g.Co, K = (long)g.N * g.P * g.Q;
  long tiles = ((M + bm - 1) / bm) * ((N + bn - 1) / bn);
  long want = (2 * 148 + tiles - 1) / tiles;
  long maxs = (K + 4 * kSimtBK - 1) / (4 * kSimtBK);
  long s = want < 1 ? 1 : (want > maxs ? maxs : want);
  long chunk = (K + s - 1) / s;
  chunk = (chunk + kSimtBK - 1) / kSimtBK * kSimtBK;
  *splits = (int)((K + chunk - 1) / chunk);
  *k_chunk = (int)chunk;
}

// Tile choice by GEMM-N (c_out for FPROP/WGRAD, c_in for DGRAD).
template <typename T, int MODE>
inline cudaError_t launch_conv_simt(cudaStream_t st, const ConvGeom& g, const T* act, const T* wgt, T* out,
                                    float* wpartial, float* wgrad_out, const T* res, const T* res_mask,
                                    uint64_t* launches) {
  long Mdim, Ndim;
  if (MODE == CONV_FPROP) { Mdim = (long)g.N * g.P * g.Q; Ndim = g.Co; }
  else if (MODE == CONV_DGRAD) { Mdim = (long)g.N * g.H * g.W; Ndim = g.Ci; }
  else { Mdim = (long)g.R * g.S * g.Ci; Ndim = g.Co; }
  int splits = 1, k_chunk = 0;
  auto go = [&](auto bm_c, auto bn_c, auto tm_c, auto tn_c) {
    constexpr int BM = decltype(bm_c)::value, BN = decltype(bn_c)::value;
    constexpr int TM = decltype(tm_c)::value, TN = decltype(tn_c)::value;
    if (MODE == CONV_WGRAD) wgrad_split(g, BM, BN, &splits, &k_chunk);
    dim3 grid((unsigned)((Mdim + BM - 1) / BM), (unsigned)((Ndim + BN - 1) / BN), (unsigned)splits);
    float* part = (MODE == CONV_WGRAD && splits == 1) ? wgrad_out : wpartial;
    conv_simt_kernel<T, MODE, BM, BN, TM, TN><<<grid, kSimtThreads, 0, st>>>(g, act, wgt, out, part, res, res_mask, k_chunk);
  };
  using std::integral_constant;
  if (Ndim <= 16) go(integral_constant<int, 128>{}, integral_constant<int, 16>{}, integral_constant<int, 4>{}, integral_constant<int, 2>{});
  else if (Ndim <= 32) go(integral_constant<int, 128>{}, integral_constant<int, 32>{}, integral_constant<int, 4>{}, integral_constant<int, 4>{});
  else go(integral_constant<int, 64>{}, integral_constant<int, 64>{}, integral_constant<int, 4>{}, integral_constant<int, 4>{});
  ++*launches;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (MODE == CONV_WGRAD && splits > 1) {
    ++*launches;
    size_t n = (size_t)Mdim * Ndim;
    e = launch_wgrad_reduce(st, wpartial, wgrad_out, n, splits);
  }
  return e;
}

// ---- weight gradient of a 3x3 / stride 1 / pad 1 convolution with very few input channels ----
// (the stem: 3 image channels).  The GEMM view has M = 9*Ci <= 36 rows against 128-row tiles, so
// the tiled kernel above spends its time gathering.  Here a block takes one image, stages strips of
// x (with its one-pixel border, zero outside the image) and dy in shared memory as floats, and
// thread (m, co) with m = (r*3+s)*Ci + ci accumulates dW[co][r][s][ci] over the strip's pixels.
// Partial sums: partial[image][co*9*Ci + m], added over the images afterwards in image order.
constexpr int kSmallWgradRows = 8;        // output rows per strip
inline bool small_wgrad_eligible(const ConvGeom& g) {
  return g.R == 3 && g.S == 3 && g.stride == 1 && g.pad == 1 && g.P == g.H && g.Q == g.W && g.Ci <= 4 &&
         9 * g.Ci * g.Co <= 1024 && g.W <= 64 &&
         ((size_t)(kSmallWgradRows + 2) * (g.W + 2) * g.Ci + (size_t)kSmallWgradRows * g.W * g.Co) * 4 <= 48 * 1024;
}
template <typename T>
__global__ void small_wgrad_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ partial,
                                   int H, int W, int Ci, int Co) {
  extern __shared__ float sw_smem[];
  const int Wp = W + 2;
  float* xs = sw_smem;                                          // [kSmallWgradRows + 2][Wp][Ci]
  float* ds = sw_smem + (kSmallWgradRows + 2) * Wp * Ci;          // [kSmallWgradRows][W][Co]
  const int n = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
  const int outs = 9 * Ci * Co;
  const int co = tid % Co, m = tid / Co, tap = m / Ci, ci = m - tap * Ci, r = tap / 3, sx = tap - 3 * r;
  const T* xn = x + (size_t)n * H * W * Ci;
  const T* dn = dy + (size_t)n * H * W * Co;
  double acc = 0.0;                       // a row's products in fp32, the rows in fp64: this gradient is compared at 1e-4
  for (int h0 = 0; h0 < H; h0 += kSmallWgradRows) {
    const int rows = min(kSmallWgradRows, H - h0);
    __syncthreads();
    for (int i = tid; i < (rows + 2) * Wp * Ci; i += nt) {
      const int c = i % Ci, w = (i / Ci) % Wp - 1, h = h0 + i / (Ci * Wp) - 1;
      xs[i] = (h >= 0 && h < H && w >= 0 && w < W) ? to_f(xn[((size_t)h * W + w) * Ci + c]) : 0.f;
    }
    for (int i = tid; i < rows * W * Co; i += nt) ds[i] = to_f(dn[(size_t)h0 * W * Co + i]);
    __syncthreads();
    if (tid < outs)
      for (int p = 0; p < rows; ++p) {
        const float* xr = xs + ((p + r) * Wp + sx) * Ci + ci;
        const float* dr = ds + (size_t)p * W * Co + co;
        float row = 0.f;
        for (int q = 0; q < W; ++q) row += xr[q * Ci] * dr[q * Co];
        acc += (double)row;
      }
  }
  if (tid < outs) partial[(size_t)n * outs + (size_t)co * 9 * Ci + m] = (float)acc;
}
// dw[Co][3][3][Ci] from x [N][H][W][Ci] and dy [N][H][W][Co]; `scratch` holds N * 9*Ci*Co floats.
template <typename T>
inline cudaError_t launch_small_wgrad(cudaStream_t st, const ConvGeom& g, const T* x, const T* dy, float* scratch,
                                      float* dw, uint64_t* launches) {
  const int outs = 9 * g.Ci * g.Co;
  const int threads = (outs + 31) / 32 * 32;
  const size_t smem = ((size_t)(kSmallWgradRows + 2) * (g.W + 2) * g.Ci + (size_t)kSmallWgradRows * g.W * g.Co) * 4;
  small_wgrad_kernel<T><<<g.N, threads, smem, st>>>(x, dy, scratch, g.H, g.W, g.Ci, g.Co);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  *launches += 2;
  return launch_wgrad_reduce(st, scratch, dw, (size_t)outs, g.N);
}

// ---- weight gradient of a 1x1 convolution (projection shortcut), stride 1 or 2, few channels ----
// dW[co][ci] = sum over output pixels of dy[n,p,q,co] * x[n,p*stride,q*stride,ci]: a Ci x Co matrix
// (512 or 2048 entries on the 6n+2 networks) from tens of thousands of pixels.  Same scheme as above:
// one image per block, strips staged in shared memory, thread (ci, co) with consecutive co in a warp.
inline bool proj_wgrad_eligible(const ConvGeom& g) {
  return g.R == 1 && g.S == 1 && g.pad == 0 && (g.stride == 1 || g.stride == 2) && g.Ci * g.Co <= 4096 && g.Co % 32 == 0 &&
         (size_t)g.Q * (g.Ci + g.Co) * 4 <= 48 * 1024;
}
// output rows per strip: what fits 48 KiB of shared memory, at most kSmallWgradRows
inline int proj_wgrad_strip(const ConvGeom& g) {
  const int fit = (int)((48 * 1024) / ((size_t)g.Q * (g.Ci + g.Co) * 4));
  return fit < kSmallWgradRows ? fit : kSmallWgradRows;
}
template <typename T>
__global__ void proj_wgrad_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ partial,
                                  int H, int W, int P, int Q, int Ci, int Co, int stride, int strip) {
  extern __shared__ float pw_smem[];
  float* xs = pw_smem;                                      // [strip][Q][Ci]
  float* ds = pw_smem + strip * Q * Ci;                     // [strip][Q][Co]
  const int n = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
  const int outs = Ci * Co;
  const T* xn = x + (size_t)n * H * W * Ci;
  const T* dn = dy + (size_t)n * P * Q * Co;
  double acc[4] = {0.0, 0.0, 0.0, 0.0};                     // thread tid owns outputs tid, tid + nt, ... (if any)
  for (int p0 = 0; p0 < P; p0 += strip) {
    const int rows = min(strip, P - p0);
    __syncthreads();
    for (int i = tid; i < rows * Q * Ci; i += nt) {
      const int c = i % Ci, q = (i / Ci) % Q, p = p0 + i / (Ci * Q);
      xs[i] = to_f(xn[((size_t)(p * stride) * W + q * stride) * Ci + c]);
    }
    for (int i = tid; i < rows * Q * Co; i += nt) ds[i] = to_f(dn[(size_t)p0 * Q * Co + i]);
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int o = tid + k * nt;
      if (o >= outs) break;
      const int co = o % Co, ci = o / Co;
      for (int p = 0; p < rows; ++p) {
        const float* xr = xs + (size_t)p * Q * Ci + ci;
        const float* dr = ds + (size_t)p * Q * Co + co;
        float row = 0.f;
        for (int q = 0; q < Q; ++q) row += xr[q * Ci] * dr[q * Co];
        acc[k] += (double)row;
      }
    }
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int o = tid + k * nt;
    if (o < outs) partial[(size_t)n * outs + (size_t)(o % Co) * Ci + o / Co] = (float)acc[k];
  }
}
template <typename T>
inline cudaError_t launch_proj_wgrad(cudaStream_t st, const ConvGeom& g, const T* x, const T* dy, float* scratch,
                                     float* dw, uint64_t* launches) {
  const int outs = g.Ci * g.Co;
  const int threads = outs >= 1024 ? 1024 : (outs + 31) / 32 * 32;
  const int strip = proj_wgrad_strip(g);
  const size_t smem = (size_t)strip * g.Q * (g.Ci + g.Co) * 4;
  proj_wgrad_kernel<T><<<g.N, threads, smem, st>>>(x, dy, scratch, g.H, g.W, g.P, g.Q, g.Ci, g.Co, g.stride, strip);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  *launches += 2;
  return launch_wgrad_reduce(st, scratch, dw, (size_t)outs, g.N);
}

// Upper bound of the fp32 scratch elements a weight-gradient launch may need.
inline size_t wgrad_scratch_elems(const ConvGeom& g) {
  long Ndim = g.Co;
  int bm = Ndim <= 32 ? 128 : 64, bn = Ndim <= 16 ? 16 : (Ndim <= 32 ? 32 : 64);
  int splits, chunk;
  wgrad_split(g, bm, bn, &splits, &chunk);
  size_t n = (size_t)splits * g.R * g.S * g.Ci * g.Co;
  if (small_wgrad_eligible(g)) n = std::max(n, (size_t)g.N * 9 * g.Ci * g.Co);
  if (proj_wgrad_eligible(g)) n = std::max(n, (size_t)g.N * g.Ci * g.Co);
  return n;
}

}  // namespace fdg
