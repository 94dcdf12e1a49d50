// Chooses the kernel for one convolution: the tcgen05 tensor-core kernels for bf16 3x3
// stride-1 convolutions whose shape they cover, the CUDA-core implicit GEMM otherwise.
#pragma once
#include <algorithm>
#include <cstring>
#include <map>
#include <vector>

#include "conv_simt.cuh"
#include "conv_tc.cuh"
#include "conv_halo.cuh"
#include "wgrad_wide.cuh"
#include "elementwise.cuh"

namespace fdg {

typedef __nv_bfloat16 bf16_t;

// Tensor maps are pure functions of (pointer, shape, box); the runtime cycles through a
// fixed set of buffers, so they are encoded once and looked up afterwards.
struct TensorMapCache {
  struct Key {
    const void* ptr; int d[8];
    bool operator<(const Key& o) const { return std::memcmp(this, &o, sizeof(Key)) < 0; }
  };
  std::map<Key, CUtensorMap> maps;
  int sm_count = 0;
  int share = 1;        // kernels expected to run side by side (one per module stream): a launch takes
                        // about sm_count / share CTAs and walks its tiles with them
  int wgrad_side_cap = 0;   // upper bound of the pixel split of a weight gradient issued beside the stream that
                            // needs its inputs' other consumers (0 = none), see halo::wgrad_ctas
};

inline bool tc_eligible(const ConvGeom& g) {
  return g.R == 3 && g.S == 3 && g.stride == 1 && g.pad == 1 && g.P == g.H && g.Q == g.W &&
         tc::conv_tc_supported(g.N, g.H, g.W, g.Ci, g.Co);
}

// Runs D = conv3x3(act, wgt) on the tensor cores.  `Ck`/`Cn` are the GEMM-K and GEMM-N channel
// counts (forward: Ci/Co; data gradient: Co/Ci with the flipped weight copy).
inline cudaError_t run_conv_tc(cudaStream_t st, TensorMapCache* cache, int N, int H, int W, int Ck, int Cn,
                               const bf16_t* act, const bf16_t* wgt, bf16_t* out, const bf16_t* res,
                               const bf16_t* res_mask, int* err_dev, int sub = 1, int taps = 9, int act_sub = 1,
                               float* stat_partial = nullptr, int* ctas_out = nullptr) {
  if (cache->sm_count == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&cache->sm_count, cudaDevAttrMultiProcessorCount, dev);
  }
  tc::ConvTcParams p = tc::conv_tc_params(N, H, W, Ck, Cn, taps);
  p.sub = sub;
  p.act_sub = act_sub;
  TensorMapCache::Key ka, kb;
  std::memset(&ka, 0, sizeof(ka)); std::memset(&kb, 0, sizeof(kb));
  ka.ptr = act; ka.d[0] = 1; ka.d[1] = N; ka.d[2] = H; ka.d[3] = W; ka.d[4] = Ck; ka.d[5] = p.kc; ka.d[6] = p.patch; ka.d[7] = act_sub;
  kb.ptr = wgt; kb.d[0] = 2; kb.d[1] = Ck; kb.d[2] = Cn; kb.d[3] = p.kc; kb.d[4] = p.n_tile; kb.d[5] = taps;
  auto ia = cache->maps.find(ka), ib = cache->maps.find(kb);
  if (ia == cache->maps.end() || ib == cache->maps.end()) {
    CUtensorMap ma, mb;
    cudaError_t e = tc::conv_tc_make_maps(p, act, wgt, &ma, &mb);
    if (e != cudaSuccess) return e;
    ia = cache->maps.insert({ka, ma}).first;
    ib = cache->maps.insert({kb, mb}).first;
  }
  return tc::conv_tc_launch(st, p, ia->second, ib->second, out, res, res_mask, err_dev, cache->sm_count, stat_partial, ctas_out);
}


// ---- halo-tile kernels (16/32/64-channel layers) ------------------------------------------
inline int cached_sm_count(TensorMapCache* cache) {
  if (cache->sm_count == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&cache->sm_count, cudaDevAttrMultiProcessorCount, dev);
  }
  return cache->sm_count;
}

inline bool halo_shape(const ConvGeom& g) {
  return g.R == 3 && g.S == 3 && g.stride == 1 && g.pad == 1 && g.P == g.H && g.Q == g.W;
}
// forward: K channels = Ci, N channels = Co; data gradient: the other way round
inline bool halo_fprop_eligible(const ConvGeom& g) { return halo_shape(g) && halo::fwd_supported(g.N, g.H, g.W, g.Ci, g.Co); }
inline bool halo_dgrad_eligible(const ConvGeom& g) { return halo_shape(g) && halo::fwd_supported(g.N, g.H, g.W, g.Co, g.Ci); }
inline bool halo_wgrad_eligible(const ConvGeom& g) { return halo_shape(g) && halo::wgrad_supported(g.N, g.H, g.W, g.Ci, g.Co); }

// A 3x3 / stride 2 / pad 1 convolution on even image sizes is the stride-1 convolution kept at the
// even pixels, and its two gradients are the stride-1 ones taken with dy spread onto the even
// pixels of a zero tensor of the input's size.  Four times the arithmetic, on kernels that are far
// from arithmetic-bound; the shapes concerned are two layers of a 6n+2 network.
inline bool halo_s2_shape(const ConvGeom& g) {
  return g.R == 3 && g.S == 3 && g.stride == 2 && g.pad == 1 && g.H % 2 == 0 && g.W % 2 == 0 && g.P == g.H / 2 && g.Q == g.W / 2;
}
inline bool halo_s2_fprop_eligible(const ConvGeom& g) { return halo_s2_shape(g) && halo::fwd_supported(g.N, g.H, g.W, g.Ci, g.Co); }
inline bool halo_s2_dgrad_eligible(const ConvGeom& g) { return halo_s2_shape(g) && halo::fwd_supported(g.N, g.H, g.W, g.Co, g.Ci); }
// the same for layers too wide for the halo kernel: the per-tap kernel at full resolution
inline bool tc_s2_fprop_eligible(const ConvGeom& g) { return halo_s2_shape(g) && tc::conv_tc_supported(g.N, g.H, g.W, g.Ci, g.Co); }
inline bool tc_s2_dgrad_eligible(const ConvGeom& g) { return halo_s2_shape(g) && tc::conv_tc_supported(g.N, g.H, g.W, g.Co, g.Ci); }
inline bool halo_s2_wgrad_eligible(const ConvGeom& g) { return halo_s2_shape(g) && halo::wgrad_supported(g.N, g.H, g.W, g.Ci, g.Co); }
// 1x1 convolutions without padding (projection shortcuts), stride 1 or 2: one "tap" of the per-tap kernel on the output
// grid; a stride-2 forward reads the even pixels of x as a strided tensor, a stride-2 data gradient writes dx at the
// even pixels (dx is cleared first).
inline bool tc_1x1_shape(const ConvGeom& g) {
  return g.R == 1 && g.S == 1 && g.pad == 0 && (g.stride == 1 || (g.stride == 2 && g.H % 2 == 0 && g.W % 2 == 0)) &&
         g.P == g.H / g.stride && g.Q == g.W / g.stride;
}
inline bool tc_1x1_fprop_eligible(const ConvGeom& g) { return tc_1x1_shape(g) && tc::conv_tc_supported(g.N, g.P, g.Q, g.Ci, g.Co); }
inline bool tc_1x1_dgrad_eligible(const ConvGeom& g) { return tc_1x1_shape(g) && tc::conv_tc_supported(g.N, g.P, g.Q, g.Co, g.Ci); }
// wide layers: the exact-tile weight-gradient kernel (stride 2 with dy spread onto the input grid; 1x1 filters on the output grid)
// (layers under 128 channels stay with the halo-tile kernel where it covers them)
inline bool wide_wgrad_eligible(const ConvGeom& g) {
  return halo_shape(g) && wide::wide_supported(g.N, g.H, g.W, g.Ci, g.Co) && ((g.Ci >= 128 && g.Co >= 128) || !halo_wgrad_eligible(g));
}
inline bool wide_s2_wgrad_eligible(const ConvGeom& g) {
  return halo_s2_shape(g) && wide::wide_supported(g.N, g.H, g.W, g.Ci, g.Co) && ((g.Ci >= 128 && g.Co >= 128) || !halo_s2_wgrad_eligible(g));
}
inline bool wide_1x1_wgrad_eligible(const ConvGeom& g) { return tc_1x1_shape(g) && wide::wide_supported(g.N, g.P, g.Q, g.Ci, g.Co, 1); }

inline cudaError_t cached_tile_map(TensorMapCache* cache, const void* act, int N, int H, int W, int C, int G,
                                   const CUtensorMap** out, int boxC = 0) {
  if (boxC == 0) boxC = C;
  TensorMapCache::Key k;
  std::memset(&k, 0, sizeof(k));
  k.ptr = act; k.d[0] = 3; k.d[1] = N; k.d[2] = H; k.d[3] = W; k.d[4] = C; k.d[5] = G; k.d[6] = boxC;
  auto it = cache->maps.find(k);
  if (it == cache->maps.end()) {
    CUtensorMap m;
    cudaError_t e = halo::make_tile_map(act, N, H, W, C, G, &m, boxC);
    if (e != cudaSuccess) return e;
    it = cache->maps.insert({k, m}).first;
  }
  *out = &it->second;
  return cudaSuccess;
}
inline cudaError_t cached_weight_map(TensorMapCache* cache, const void* wgt, int Ck, int Cn, const CUtensorMap** out) {
  TensorMapCache::Key k;
  std::memset(&k, 0, sizeof(k));
  k.ptr = wgt; k.d[0] = 4; k.d[1] = Ck; k.d[2] = Cn;
  auto it = cache->maps.find(k);
  if (it == cache->maps.end()) {
    CUtensorMap m;
    cudaError_t e = halo::make_weight_map(wgt, Ck, Cn, &m);
    if (e != cudaSuccess) return e;
    it = cache->maps.insert({k, m}).first;
  }
  *out = &it->second;
  return cudaSuccess;
}

// out = conv3x3(act, wgt) [+ res * [mask > 0]]; act [N][H][W][Ck], wgt [Cn][9*Ck], out [N][H][W][Cn].
// `red` (nullable, Cn <= 64 only) asks for a per-channel reduction in the epilogue; its `partial`
// must hold 2*Cn floats per CTA; *ctas_out receives the number of CTAs, i.e. of partial rows.
inline bool halo_reduce_ok(int Cn) { return Cn <= 64; }
inline cudaError_t run_conv_halo(cudaStream_t st, TensorMapCache* cache, int N, int H, int W, int Ck, int Cn,
                                 const bf16_t* act, const bf16_t* wgt, bf16_t* out, const bf16_t* res,
                                 const bf16_t* res_mask, int* err_dev, const halo::EpiReduce* red = nullptr,
                                 int* ctas_out = nullptr, int sub = 1) {
  int sms = cached_sm_count(cache) / (cache->share > 0 ? cache->share : 1);
  if (sms < 16) sms = 16;
  halo::FwdParams p = halo::fwd_params(N, H, W, Ck, Cn, sms);
  p.sub = sub;
  const CUtensorMap *mx, *mw;
  cudaError_t e = cached_tile_map(cache, act, N, H, W, Ck, p.G, &mx);
  if (e == cudaSuccess) e = cached_weight_map(cache, wgt, Ck, Cn, &mw);
  if (e == cudaSuccess) e = halo::set_smem_attrs();
  if (e != cudaSuccess) return e;
  // the fewest CTAs that keep the number of tiles of the busiest one at ceil(tiles / sms)
  const int per_cta = (p.tiles + sms - 1) / sms;
  const int grid = (p.tiles + per_cta - 1) / per_cta;
  halo::EpiReduce r{};
  if (red) { if (!halo_reduce_ok(Cn)) return cudaErrorInvalidValue; r = *red; }
  if (ctas_out) *ctas_out = grid;
  return launch_chained(halo::conv_halo_kernel, grid, halo::kConvThreads, halo::fwd_smem_bytes(p), st, *mx, *mw, p, out, res, res_mask, r, err_dev);
}

// dw[Co][3][3][Ci] (fp32) from x [N][H][W][Ci] and dy [N][H][W][Co]; `scratch` holds the per-CTA partials
// (halo::wgrad_scratch_elems floats).  Two launches: the tensor-core kernel and the fixed-order sum.
inline cudaError_t run_wgrad_halo(cudaStream_t st, TensorMapCache* cache, int N, int H, int W, int Ci, int Co,
                                  const bf16_t* x, const bf16_t* dy, float* dw, float* scratch, int* err_dev,
                                  bool side = false) {
  halo::WgradParams p = halo::wgrad_params(N, H, W, Ci, Co);
  const CUtensorMap *mx, *my;
  cudaError_t e = cached_tile_map(cache, x, N, H, W, Ci, p.G, &mx, p.kcx);
  if (e == cudaSuccess) e = cached_tile_map(cache, dy, N, H, W, Co, p.G, &my, p.kcy);
  if (e == cudaSuccess) e = halo::set_smem_attrs();
  if (e != cudaSuccess) return e;
  const int ctas = halo::wgrad_ctas(p, side ? cache->wgrad_side_cap : 0);
  halo::wgrad_halo_kernel<<<dim3(ctas, halo::wgrad_pairs(p)), halo::kFwdThreads, halo::wgrad_smem_bytes(p), st>>>(*mx, *my, p, scratch, err_dev);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const size_t n = (size_t)Co * 9 * Ci;
  if (n >= ((size_t)1 << 17) && ctas <= 8)        // large filters, few partials: four outputs per thread, partials in turn
    wide::wgrad_wide_sum_kernel<<<(unsigned)((n / 4 + 255) / 256), 256, 0, st>>>(reinterpret_cast<const float4*>(scratch),
                                                                               reinterpret_cast<float4*>(dw), n / 4, ctas);
  else
    halo::wgrad_halo_reduce_kernel<<<(int)((n + 31) / 32), 256, 0, st>>>(scratch, dw, n, ctas);
  return cudaGetLastError();
}

// The same contract for wide layers and 1x1 filters (wide::wgrad_wide_kernel; scratch of wide::wide_scratch_elems
// floats).  R = 1: H, W are the output grid and `x_sub` the stride (2: x is [N][2H][2W][Ci], read at its even pixels).
inline cudaError_t cached_slab_map(TensorMapCache* cache, const void* act, int N, int H, int W, int C, int box_w, int box_h,
                                   const CUtensorMap** out, int sub = 1) {
  TensorMapCache::Key k;
  std::memset(&k, 0, sizeof(k));
  k.ptr = act; k.d[0] = 5; k.d[1] = N; k.d[2] = H; k.d[3] = W; k.d[4] = C; k.d[5] = box_w; k.d[6] = box_h; k.d[7] = sub;
  auto it = cache->maps.find(k);
  if (it == cache->maps.end()) {
    CUtensorMap m;
    cudaError_t e = wide::make_slab_map(act, N, H, W, C, box_w, box_h, &m, sub);
    if (e != cudaSuccess) return e;
    it = cache->maps.insert({k, m}).first;
  }
  *out = &it->second;
  return cudaSuccess;
}
inline cudaError_t run_wgrad_wide(cudaStream_t st, TensorMapCache* cache, int N, int H, int W, int Ci, int Co,
                                  const bf16_t* x, const bf16_t* dy, float* dw, float* scratch, int* err_dev, int R = 3,
                                  int x_sub = 1) {
  const wide::WideParams p = wide::wide_params(N, H, W, Ci, Co, cached_sm_count(cache), R);
  const CUtensorMap *mx, *my;
  cudaError_t e = cached_slab_map(cache, x, N, H, W, Ci, p.xw, p.S, &mx, x_sub);
  if (e == cudaSuccess) e = cached_slab_map(cache, dy, N, H, W, Co, p.W, p.S, &my);
  if (e == cudaSuccess) e = wide::wide_set_attrs();
  if (e != cudaSuccess) return e;
  const dim3 grid(p.co_blocks * p.ci_chunks * p.rdim, p.splits);
  if (R == 3) wide::wgrad_wide_kernel<3><<<grid, wide::kWideThreads, wide::wide_smem_bytes(p), st>>>(*mx, *my, p, scratch, err_dev);
  else wide::wgrad_wide_kernel<1><<<grid, wide::kWideThreads, wide::wide_smem_bytes(p), st>>>(*mx, *my, p, scratch, err_dev);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const size_t n4 = (size_t)Co * R * R * Ci / 4;                 // Ci is a multiple of 16
  // the sum's launch overlaps the tail of the kernel above; it waits for that kernel before it reads
  return launch_chained(wide::wgrad_wide_sum_kernel, dim3((unsigned)((n4 + 255) / 256)), dim3(256), 0, st,
                        reinterpret_cast<const float4*>(scratch), reinterpret_cast<float4*>(dw), n4, p.splits);
}

// Does the data gradient of this convolution read the flipped/transposed weight copy?
inline bool dgrad_uses_flipped(const ConvGeom& g) {
  return halo_dgrad_eligible(g) || halo_s2_dgrad_eligible(g) || tc_eligible(g) || tc_s2_dgrad_eligible(g) || tc_1x1_dgrad_eligible(g);
}
// Do the stride-2 gradients of this convolution run on the tensor cores, given a spread-out copy of dy?
inline bool s2_uses_spread_dy(const ConvGeom& g) {
  return (halo_s2_dgrad_eligible(g) || halo_s2_wgrad_eligible(g) || tc_s2_dgrad_eligible(g) || wide_s2_wgrad_eligible(g)) && g.Co % 8 == 0;
}

// fp32 scratch elements a weight-gradient call may need (bf16 storage: whichever kernel is chosen).
inline size_t conv_wgrad_scratch_elems(bool bf16_storage, const ConvGeom& g) {
  size_t n = wgrad_scratch_elems(g);
  if (bf16_storage && (halo_wgrad_eligible(g) || halo_s2_wgrad_eligible(g)))
    n = std::max(n, halo::wgrad_scratch_elems(g.N, g.H, g.W, g.Ci, g.Co));
  if (bf16_storage && (wide_wgrad_eligible(g) || wide_s2_wgrad_eligible(g)))
    n = std::max(n, wide::wide_scratch_elems(g.N, g.H, g.W, g.Ci, g.Co));
  if (bf16_storage && wide_1x1_wgrad_eligible(g))
    n = std::max(n, wide::wide_scratch_elems(g.N, g.P, g.Q, g.Ci, g.Co, 1));
  return n;
}

// ---- one convolution operator in bf16 storage: which kernel, in which launch shape ------------------
// Used by the module runtime and by the operator-level entry points alike.  `launches` counts kernels.

// dy [N][P][Q][Co] of a stride-2 convolution spread onto the even pixels of a zero [N][H][W][Co] tensor `up`.
inline cudaError_t bf16_spread_dy(cudaStream_t st, const ConvGeom& g, const bf16_t* dy, bf16_t* up, uint64_t* launches) {
  const size_t nvec = (size_t)g.N * g.H * g.W * g.Co / 8;
  upsample2_kernel<bf16_t, 8><<<ew_blocks(nvec), 256, 0, st>>>(dy, up, nvec, g.P, g.Q, g.Co);
  ++*launches;
  return cudaGetLastError();
}

// y = conv(x, w) [+ res].  `red` (mode 1) asks for the per-CTA sums of y and y^2; *nparts receives the number
// of rows left in red->partial, 0 when the chosen kernel forms none.
// Where the statistics of y go when a wide layer's kernel forms their partial sums (WideStats): `partial` holds one
// row of 2 * Co floats per CTA; with `stats` set, the totals are finalised right behind the convolution (mean and
// 1/sqrt(var + eps) over `rows` values per channel, running statistics included) and *nparts = -1 tells the caller
// that nothing is left to do; without, *nparts = the rows left in `partial`.
struct WideStats {
  float* partial; size_t partial_floats;
  float* stats; size_t rows; float eps;
  float* running; float momentum;
};
inline bool wide_stats_ok(TensorMapCache* cache, const ConvGeom& g, const WideStats* ws) {
  return ws && ws->partial && g.Co <= tc::kStatChunks * 16 && (size_t)cached_sm_count(cache) * 2 * g.Co <= ws->partial_floats;
}
inline cudaError_t finish_wide_stats(cudaStream_t st, const ConvGeom& g, const WideStats* ws, int ctas, int* nparts,
                                     uint64_t* launches) {
  if (!ws->stats) { if (nparts) *nparts = ctas; return cudaSuccess; }
  const RunningStats run{ws->running, ws->momentum, ws->rows > 1 ? (float)((double)ws->rows / (double)(ws->rows - 1)) : 1.f};
  ++*launches;
  if (nparts) *nparts = -1;
  return launch_chained(stats_finalize_kernel, dim3((unsigned)((g.Co + 31) / 32)), dim3(256), 0, st, (const float*)ws->partial, ctas,
                        g.Co, 1.0 / (double)ws->rows, ws->eps, ws->stats, run);
}

inline cudaError_t bf16_conv_fprop(cudaStream_t st, TensorMapCache* cache, const ConvGeom& g, const bf16_t* x,
                                   const bf16_t* w, bf16_t* y, const bf16_t* res, const halo::EpiReduce* red, int* nparts,
                                   int* err_dev, uint64_t* launches, const WideStats* ws = nullptr) {
  if (nparts) *nparts = 0;
  const bool s1 = halo_fprop_eligible(g), s2 = !s1 && halo_s2_fprop_eligible(g);
  if (s1 || s2) {
    ++*launches;
    const bool fuse = red && red->mode == 1 && halo_reduce_ok(g.Co);
    int ctas = 0;
    cudaError_t e = run_conv_halo(st, cache, g.N, g.H, g.W, g.Ci, g.Co, x, w, y, res, nullptr, err_dev, fuse ? red : nullptr, &ctas, s2 ? 2 : 1);
    if (fuse && nparts) *nparts = ctas;
    return e;
  }
  if (tc_eligible(g) || tc_s2_fprop_eligible(g)) {
    ++*launches;
    if (wide_stats_ok(cache, g, ws)) {
      int ctas = 0;
      const cudaError_t e = run_conv_tc(st, cache, g.N, g.H, g.W, g.Ci, g.Co, x, w, y, res, nullptr, err_dev, g.stride, 9, 1, ws->partial, &ctas);
      return e != cudaSuccess ? e : finish_wide_stats(st, g, ws, ctas, nparts, launches);
    }
    return run_conv_tc(st, cache, g.N, g.H, g.W, g.Ci, g.Co, x, w, y, res, nullptr, err_dev, g.stride);
  }
  if (tc_1x1_fprop_eligible(g)) {
    ++*launches;
    if (wide_stats_ok(cache, g, ws)) {
      int ctas = 0;
      const cudaError_t e = run_conv_tc(st, cache, g.N, g.P, g.Q, g.Ci, g.Co, x, w, y, res, nullptr, err_dev, 1, 1, g.stride, ws->partial, &ctas);
      return e != cudaSuccess ? e : finish_wide_stats(st, g, ws, ctas, nparts, launches);
    }
    return run_conv_tc(st, cache, g.N, g.P, g.Q, g.Ci, g.Co, x, w, y, res, nullptr, err_dev, 1, 1, g.stride);
  }
  return launch_conv_simt<bf16_t, CONV_FPROP>(st, g, x, w, y, nullptr, nullptr, res, (const bf16_t*)nullptr, launches);
}

// dx = conv^T(dy, w) [+ res * [mask > 0]].  `wflip` is the flipped/transposed weight copy (null: CUDA cores);
// `dy_up` the spread-out dy of a stride-2 layer (null: its gradient stays on the CUDA cores).  `red` (mode 2)
// asks for the sums of the batch-norm backward that dx feeds.
inline cudaError_t bf16_conv_dgrad(cudaStream_t st, TensorMapCache* cache, const ConvGeom& g, const bf16_t* dy,
                                   const bf16_t* w, const bf16_t* wflip, const bf16_t* dy_up, bf16_t* dx, const bf16_t* res,
                                   const bf16_t* mask, const halo::EpiReduce* red, int* nparts, int* err_dev,
                                   uint64_t* launches) {
  if (nparts) *nparts = 0;
  const bool h1 = wflip && halo_dgrad_eligible(g), h2 = !h1 && wflip && dy_up && halo_s2_dgrad_eligible(g);
  if (h1 || h2) {
    ++*launches;
    const bool fuse = red && red->mode == 2 && halo_reduce_ok(g.Ci);
    int ctas = 0;
    cudaError_t e = run_conv_halo(st, cache, g.N, g.H, g.W, g.Co, g.Ci, h1 ? dy : dy_up, wflip, dx, res, mask, err_dev, fuse ? red : nullptr, &ctas);
    if (fuse && nparts) *nparts = ctas;
    return e;
  }
  if (wflip && tc_eligible(g)) {
    ++*launches;
    return run_conv_tc(st, cache, g.N, g.H, g.W, g.Co, g.Ci, dy, wflip, dx, res, mask, err_dev);
  }
  if (wflip && dy_up && tc_s2_dgrad_eligible(g)) {
    ++*launches;
    return run_conv_tc(st, cache, g.N, g.H, g.W, g.Co, g.Ci, dy_up, wflip, dx, res, mask, err_dev);
  }
  if (wflip && tc_1x1_dgrad_eligible(g) && (g.stride == 1 || (!res && !mask))) {
    // stride 2: only the even pixels of dx receive a gradient; the rest of dx is cleared first
    if (g.stride == 2) {
      const cudaError_t e = cudaMemsetAsync(dx, 0, (size_t)g.N * g.H * g.W * g.Ci * sizeof(bf16_t), st);
      if (e != cudaSuccess) return e;
    }
    ++*launches;
    return run_conv_tc(st, cache, g.N, g.P, g.Q, g.Co, g.Ci, dy, wflip, dx, res, mask, err_dev, g.stride == 2 ? 3 : 1, 1, 1);
  }
  return launch_conv_simt<bf16_t, CONV_DGRAD>(st, g, dy, w, dx, nullptr, nullptr, res, mask, launches);
}

// dw (fp32) from x and dy; `scratch` of conv_wgrad_scratch_elems floats; `side`: bound the pixel split by
// cache->wgrad_side_cap (a weight gradient issued beside the chain that needs the SMs more).
inline cudaError_t bf16_conv_wgrad(cudaStream_t st, TensorMapCache* cache, const ConvGeom& g, const bf16_t* x,
                                   const bf16_t* dy, const bf16_t* dy_up, float* dw, float* scratch, int* err_dev,
                                   bool side, uint64_t* launches) {
  if ((dy_up && wide_s2_wgrad_eligible(g)) || wide_wgrad_eligible(g)) {
    *launches += 2;
    return run_wgrad_wide(st, cache, g.N, g.H, g.W, g.Ci, g.Co, x, wide_wgrad_eligible(g) ? dy : dy_up, dw, scratch, err_dev);
  }
  if (wide_1x1_wgrad_eligible(g)) {
    *launches += 2;
    return run_wgrad_wide(st, cache, g.N, g.P, g.Q, g.Ci, g.Co, x, dy, dw, scratch, err_dev, 1, g.stride);
  }
  if (dy_up && halo_s2_wgrad_eligible(g)) {
    *launches += 2;
    return run_wgrad_halo(st, cache, g.N, g.H, g.W, g.Ci, g.Co, x, dy_up, dw, scratch, err_dev, side);
  }
  if (halo_wgrad_eligible(g)) {
    *launches += 2;
    return run_wgrad_halo(st, cache, g.N, g.H, g.W, g.Ci, g.Co, x, dy, dw, scratch, err_dev, side);
  }
  if (small_wgrad_eligible(g)) return launch_small_wgrad<bf16_t>(st, g, x, dy, scratch, dw, launches);
  if (proj_wgrad_eligible(g)) return launch_proj_wgrad<bf16_t>(st, g, x, dy, scratch, dw, launches);
  return launch_conv_simt<bf16_t, CONV_WGRAD>(st, g, x, dy, (bf16_t*)nullptr, scratch, dw, (const bf16_t*)nullptr, (const bf16_t*)nullptr, launches);
}

}  // namespace fdg
