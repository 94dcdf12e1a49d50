// Chooses the kernel for one convolution: the tcgen05 tensor-core kernels for bf16 3x3
// stride-1 convolutions whose shape they cover, the CUDA-core implicit GEMM otherwise.
#pragma once
#include <cstring>
#include <map>
#include <vector>

#include "conv_simt.cuh"
#include "conv_tc.cuh"

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
};

inline bool tc_eligible(const ConvGeom& g) {
  return g.R == 3 && g.S == 3 && g.stride == 1 && g.pad == 1 && g.P == g.H && g.Q == g.W &&
         tc::conv_tc_supported(g.N, g.H, g.W, g.Ci, g.Co);
}

// Runs D = conv3x3(act, wgt) on the tensor cores.  `Ck`/`Cn` are the GEMM-K and GEMM-N channel
// counts (forward: Ci/Co; data gradient: Co/Ci with the flipped weight copy).
inline cudaError_t run_conv_tc(cudaStream_t st, TensorMapCache* cache, int N, int H, int W, int Ck, int Cn,
                               const bf16_t* act, const bf16_t* wgt, bf16_t* out, const bf16_t* res,
                               const bf16_t* res_mask, int* err_dev) {
  if (cache->sm_count == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&cache->sm_count, cudaDevAttrMultiProcessorCount, dev);
  }
  tc::ConvTcParams p = tc::conv_tc_params(N, H, W, Ck, Cn);
  TensorMapCache::Key ka, kb;
  std::memset(&ka, 0, sizeof(ka)); std::memset(&kb, 0, sizeof(kb));
  ka.ptr = act; ka.d[0] = 1; ka.d[1] = N; ka.d[2] = H; ka.d[3] = W; ka.d[4] = Ck; ka.d[5] = p.kc;
  kb.ptr = wgt; kb.d[0] = 2; kb.d[1] = Ck; kb.d[2] = Cn; kb.d[3] = p.kc; kb.d[4] = p.n_tile;
  auto ia = cache->maps.find(ka), ib = cache->maps.find(kb);
  if (ia == cache->maps.end() || ib == cache->maps.end()) {
    CUtensorMap ma, mb;
    cudaError_t e = tc::conv_tc_make_maps(p, act, wgt, &ma, &mb);
    if (e != cudaSuccess) return e;
    ia = cache->maps.insert({ka, ma}).first;
    ib = cache->maps.insert({kb, mb}).first;
  }
  return tc::conv_tc_launch(st, p, ia->second, ib->second, out, res, res_mask, err_dev, cache->sm_count);
}

}  // namespace fdg
