// Memory-bound kernels of the FDG module-step: batch-norm statistics / apply /
// backward, the classifier head, the shrink of the received delayed gradient
// (Eq. 15), the SGD-momentum update (Eq. 11), image ingest and dtype conversion.
//
// All tensors are NHWC, seen here as [rows = N*H*W][C].  T is the storage type
// (float or __nv_bfloat16); arithmetic, statistics and reductions are fp32 (final
// combination of per-block partial sums in fp64).  Every reduction has a fixed
// order, so results do not depend on scheduling.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace fdg {

// ------------------------------------------------ programmatic dependent launch --
// The kernels that follow one another in a module's chain (convolution, batch-norm apply, batch-norm
// backward apply) are launched with programmatic stream serialisation: the next kernel of the stream may be
// scheduled while this one still runs, does the part of its start-up that needs nothing from global
// memory (barriers, tensor-memory allocation, descriptor prefetch), and then blocks in grid_dependency_wait()
// until the preceding kernel has completed and its writes are visible.  Nothing may be read from or written
// to global memory before that wait.  grid_dependency_release() tells the scheduler that, as far as this
// block is concerned, the next kernel may start being scheduled (it fires once every block has called it or
// exited).  Both are no-ops in a kernel launched the ordinary way.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launch with the attribute that allows the overlap described above.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---------------------------------------------------------------- helpers ---
template <typename T> struct Vec;   // 16-byte vector of T
template <> struct Vec<float> {
  static constexpr int N = 4;
  float v[4];
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __nv_bfloat16 v[8];
};

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Loads VEC consecutive elements (VEC == 1 or a full 16-byte vector) as floats.
template <typename T, int VEC>
__device__ __forceinline__ void load_vec(const T* __restrict__ p, float (&out)[VEC]) {
  if constexpr (VEC == 1) {
    out[0] = to_f(p[0]);
  } else {
    static_assert(VEC * sizeof(T) == 16, "vector must be 16 bytes");
    uint4 raw = *reinterpret_cast<const uint4*>(p);
    const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
    for (int i = 0; i < VEC; ++i) out[i] = to_f(e[i]);
  }
}
template <typename T, int VEC>
__device__ __forceinline__ void store_vec(T* __restrict__ p, const float (&in)[VEC]) {
  if constexpr (VEC == 1) {
    p[0] = from_f<T>(in[0]);
  } else {
    uint4 raw;
    T* e = reinterpret_cast<T*>(&raw);
#pragma unroll
    for (int i = 0; i < VEC; ++i) e[i] = from_f<T>(in[i]);
    *reinterpret_cast<uint4*>(p) = raw;
  }
}

// Running statistics of a batch norm, kept for inference beside the batch statistics of training:
// running[0..C) mean, running[C..2C) variance; each forward folds in the batch mean and the unbiased batch
// variance with weight `momentum` (null pointer: not kept).
struct RunningStats {
  float* running;
  float momentum;
  float unbias;      // M / (M - 1) for M values per channel
};
__device__ __forceinline__ void update_running(const RunningStats& r, int C, int c, float mean, float biased_var) {
  r.running[c] = (1.f - r.momentum) * r.running[c] + r.momentum * mean;
  r.running[C + c] = (1.f - r.momentum) * r.running[C + c] + r.momentum * (biased_var * r.unbias);
}

constexpr int kRedThreads = 256;      // threads per block of the channel-reduction kernels
// Blocks of a channel reduction along the rows.  The last block of a channel slab to finish adds that slab's
// partial sums, a serial tail that grows with the block count and with the slab's width; wide tensors are
// therefore cut into slabs of kRedSlab channels (grid.y), each with its own tail on its own SM.
constexpr int kRedMaxBlocks = 148;
constexpr int kRedMaxSums = 3;
constexpr int kRedSlab = 32;
constexpr int kRedMaxSlabs = 64;      // ticket words available

// Per-channel statistics record written by the forward and read by the backward.
// stats[0..C) = mean, stats[C..2C) = 1/sqrt(var+eps).

// Geometry shared by the channel-reduction kernels: a block owns a contiguous range
// of rows; thread (r, cv) walks rows r, r+RP, ... of channel vector cv.
// C: channels of one slab (what a block reduces); ld: channels of a row of the tensor; the slab of block
// (x, y) starts at channel y * C.
struct RedGeom {
  int rows, C, cv, rp, blocks, rows_per_block, ld, slabs;
};
inline RedGeom red_geom(int rows, int C, int vec) {
  RedGeom g;
  g.ld = C;
  g.slabs = 1;
  if (C > 2 * kRedSlab && C % kRedSlab == 0 && kRedSlab % vec == 0 && C / kRedSlab <= kRedMaxSlabs) { g.slabs = C / kRedSlab; C = kRedSlab; }
  g.rows = rows; g.C = C; g.cv = C / vec;
  g.rp = kRedThreads / g.cv; if (g.rp < 1) g.rp = 1;
  int want = (rows + g.rp * 4 - 1) / (g.rp * 4);           // >= 4 passes per block
  g.blocks = want < 1 ? 1 : (want > kRedMaxBlocks ? kRedMaxBlocks : want);
  g.rows_per_block = (rows + g.blocks - 1) / g.blocks;
  return g;
}

// Block-level part: NS sums per channel -> partial[block][NS][C]; the last block to
// finish adds the partials in block order (fp64) and calls `fin(c, sums[NS])`.
// The dynamic shared memory of the reduction kernels, reused as doubles for the final totals
// (NS*C doubles <= rp*NS*C floats whenever rp >= 2; the launchers reserve at least that).
__device__ __forceinline__ double* red_smem_d() {
  extern __shared__ double red_smem_as_double[];
  return red_smem_as_double;
}

template <int NS, int VEC, typename Acc, typename Fin>
__device__ __forceinline__ void channel_reduce(const RedGeom g, float* __restrict__ partial,
                                               unsigned int* __restrict__ counter, Acc acc, Fin fin_fn) {
  extern __shared__ float red_smem[];                        // [rp][NS][C]
  __shared__ bool is_last;
  const int tid = threadIdx.x;
  const int cvi = tid % g.cv, r = tid / g.cv;
  const int C = g.C;
  const int c_off = blockIdx.y * C;                          // first channel of this block's slab
  partial += (size_t)blockIdx.y * gridDim.x * NS * C;         // this slab's partial sums
  counter += blockIdx.y;
  float sums[NS][VEC];
#pragma unroll
  for (int s = 0; s < NS; ++s)
#pragma unroll
    for (int i = 0; i < VEC; ++i) sums[s][i] = 0.f;
  const int row0 = blockIdx.x * g.rows_per_block;
  const int row1 = min(row0 + g.rows_per_block, g.rows);
  if (r < g.rp) {
#pragma unroll 4
    for (int row = row0 + r; row < row1; row += g.rp) acc(row, c_off + cvi * VEC, sums);
  }
  if (r < g.rp) {
#pragma unroll
    for (int s = 0; s < NS; ++s)
#pragma unroll
      for (int i = 0; i < VEC; ++i) red_smem[(r * NS + s) * C + cvi * VEC + i] = sums[s][i];
  }
  __syncthreads();
  for (int j = tid; j < NS * C; j += blockDim.x) {
    float a = 0.f;
    for (int rr = 0; rr < g.rp; ++rr) a += red_smem[rr * NS * C + j];
    partial[(size_t)blockIdx.x * NS * C + j] = a;
  }
  // Release: the block's partial sums were written by all of its threads, the ticket is taken by one.
  // The fence that makes them visible before the ticket has to be executed by the ticket's thread
  // AFTER the barrier that orders it behind the other threads' writes: a fence each writer executes
  // before the barrier orders only that writer's own later accesses, and the ticket could then reach
  // L2 ahead of another warp's partial sums (seen on some GPUs as a last block adding stale rows).
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    is_last = (atomicInc(counter, gridDim.x - 1) == gridDim.x - 1);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();                                           // acquire: before the other blocks' partial sums are read
  // NS*C (sum, channel) pairs; kRedThreads / pairs threads share a pair, each taking every
  // nseg-th block with 8 loads in flight; the segment sums are then added in segment order.
  __shared__ double fin[kRedThreads];
  const int pairs = NS * C;
  for (int p0 = 0; p0 < pairs; p0 += kRedThreads) {
    const int np = min(pairs - p0, kRedThreads);
    const int nseg = kRedThreads / np;
    const int t = tid % np, seg = tid / np;
    double a = 0.0;
    if (seg < nseg)
      for (unsigned b0 = seg; b0 < gridDim.x; b0 += 8 * nseg) {
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const unsigned b = b0 + u * nseg;
          v[u] = b < gridDim.x ? __ldcg(&partial[(size_t)b * pairs + p0 + t]) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) a += (double)v[u];
      }
    fin[tid] = a;
    __syncthreads();
    if (tid < np) {
      double tot = 0.0;
      for (int q = 0; q < nseg; ++q) tot += fin[q * np + tid];
      red_smem_d()[p0 + tid] = tot;
    }
    __syncthreads();
  }
  for (int c = tid; c < C; c += blockDim.x) {
    double tot[NS];
#pragma unroll
    for (int s = 0; s < NS; ++s) tot[s] = red_smem_d()[s * C + c];
    fin_fn(c_off + c, tot);
  }
}

// ------------------------------------------------- batch norm, forward ------
// mean and 1/sqrt(var+eps) of each channel over all rows (biased variance).
template <typename T, int VEC>
__global__ void __launch_bounds__(kRedThreads)
bn_stats_kernel(const T* __restrict__ x, RedGeom g, float eps, float* __restrict__ stats,
                float* __restrict__ partial, unsigned int* __restrict__ counter, RunningStats run) {
  const int C = g.ld;
  const double inv_m = 1.0 / (double)g.rows;
  channel_reduce<2, VEC>(
      g, partial, counter,
      [&](int row, int c0, float (&s)[2][VEC]) {
        float v[VEC];
        load_vec<T, VEC>(x + (size_t)row * C + c0, v);
#pragma unroll
        for (int i = 0; i < VEC; ++i) { s[0][i] += v[i]; s[1][i] += v[i] * v[i]; }
      },
      [&](int c, double (&tot)[2]) {
        double mean = tot[0] * inv_m;
        double var = tot[1] * inv_m - mean * mean;
        if (var < 0.0) var = 0.0;
        stats[c] = (float)mean;
        stats[C + c] = (float)(1.0 / sqrt(var + (double)eps));
        if (run.running) update_running(run, C, c, (float)mean, (float)var);
      });
}

// Statistics from the rows of partial sums a wide convolution's epilogue left: partial[nparts][2][C] (sum, sum of
// squares per CTA) -> stats[0..C) = mean, stats[C..2C) = 1/sqrt(var + eps), and the running statistics.  A block
// takes 32 channels; its 8 warps take every 8th row, their sums are added in warp order (fp64).
__global__ void __launch_bounds__(256) stats_finalize_kernel(const float* __restrict__ partial, int nparts, int C, double inv_count,
                                                             float eps, float* __restrict__ stats, RunningStats run) {
  grid_dependency_wait();                   // launched ahead of the end of the convolution that writes `partial`
  __shared__ double fin[2][8][32];
  const int lane = threadIdx.x & 31, seg = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + lane;
  double s = 0.0, ss = 0.0;
  if (c < C)
    for (int r = seg; r < nparts; r += 8) {
      s += (double)partial[(size_t)r * 2 * C + c];
      ss += (double)partial[(size_t)r * 2 * C + C + c];
    }
  fin[0][seg][lane] = s; fin[1][seg][lane] = ss;
  __syncthreads();
  if (seg == 0 && c < C) {
    double a = 0.0, b = 0.0;
#pragma unroll
    for (int q = 0; q < 8; ++q) { a += fin[0][q][lane]; b += fin[1][q][lane]; }
    const double mean = a * inv_count;
    double var = b * inv_count - mean * mean;
    if (var < 0.0) var = 0.0;
    stats[c] = (float)mean;
    stats[C + c] = (float)(1.0 / sqrt(var + (double)eps));
    if (run.running) update_running(run, C, c, (float)mean, (float)var);
  }
}

// Per-CTA partial sums left by a convolution epilogue, partial[nparts][2*C], to be added up by
// the kernel that consumes the totals (every block does it for itself: the partials are a few KB
// and sit in L2).  Fixed order: kEwThreads / (2C) threads share a (sum, channel) pair, each taking
// every nseg-th partial with 8 loads in flight; segment sums are added in segment order.
//   kind 1  totals are (sum x, sum x^2): out2c = (mean, 1/sqrt(var + eps))
//   kind 2  totals are the batch-norm backward's (sum dz, sum dz*xhat): out2c = the totals
struct PartialSums {
  const float* partial;     // null: nothing to add up (the totals are read from global memory instead)
  int nparts;
  int kind;
  float inv_count, eps;     // kind 1
  float* save0;             // block 0 stores out2c[0..C) here (kind 1: with save1 contiguous = stats[2C]; kind 2: dbeta)
  float* save1;             // and out2c[C..2C) here (kind 2: dgamma)
  RunningStats run;         // kind 1: block 0 also folds the batch statistics into the running ones
};
constexpr int kEwThreads = 256;

// Fills out2c[2*C] (shared memory) from the partials; requires blockDim.x == kEwThreads and 2*C <= kEwThreads.
__device__ __forceinline__ void finalize_partials(const PartialSums ps, int C, float* out2c) {
  __shared__ double fin[kEwThreads];
  const int tid = threadIdx.x, pairs = 2 * C;
  const int nseg = kEwThreads / pairs;
  const int t = tid % pairs, seg = tid / pairs;
  double a = 0.0;
  if (seg < nseg)
    for (int b0 = seg; b0 < ps.nparts; b0 += 8 * nseg) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int b = b0 + u * nseg;
        v[u] = b < ps.nparts ? __ldcg(&ps.partial[(size_t)b * pairs + t]) : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) a += (double)v[u];
    }
  fin[tid] = a;
  __syncthreads();
  if (tid < C) {
    double s0 = 0.0, s1 = 0.0;
    for (int q = 0; q < nseg; ++q) { s0 += fin[q * pairs + tid]; s1 += fin[q * pairs + C + tid]; }
    float o0, o1;
    if (ps.kind == 1) {
      const double mean = s0 * (double)ps.inv_count;
      double var = s1 * (double)ps.inv_count - mean * mean;
      if (var < 0.0) var = 0.0;
      o0 = (float)mean; o1 = (float)(1.0 / sqrt(var + (double)ps.eps));
      if (blockIdx.x == 0 && ps.run.running) update_running(ps.run, C, tid, (float)mean, (float)var);
    } else {
      o0 = (float)s0; o1 = (float)s1;
    }
    out2c[tid] = o0; out2c[C + tid] = o1;
    if (blockIdx.x == 0) { ps.save0[tid] = o0; ps.save1[tid] = o1; }
  }
  __syncthreads();
}

// y = [relu]( gamma*(x-mean)*invstd + beta + residual ), residual = none | r | BN_r(r).
// The statistics come from `stats`, or are first formed from `ps.partial` (and saved to stats).
// The launcher makes the grid's thread count a multiple of the channel vectors per row, so a thread
// meets the same VEC channels in every iteration: their constants live in registers, and the loop
// keeps kEwUnroll independent 16-byte loads per operand in flight.
constexpr int kEwUnroll = 4;
// 16 raw bytes (or one element when VEC == 1) of T, converted to floats only when used, so that
// several loads can be in flight without holding their float images in registers.
template <typename T, int VEC> struct RawVec { uint4 q; };
template <typename T> struct RawVec<T, 1> { T q; };
template <typename T, int VEC> __device__ __forceinline__ RawVec<T, VEC> load_raw(const T* __restrict__ p) {
  RawVec<T, VEC> r;
  if constexpr (VEC == 1) r.q = p[0]; else r.q = *reinterpret_cast<const uint4*>(p);
  return r;
}
template <typename T, int VEC> __device__ __forceinline__ void raw_to_f(const RawVec<T, VEC>& r, float (&out)[VEC]) {
  if constexpr (VEC == 1) {
    out[0] = to_f(r.q);
  } else {
    const T* e = reinterpret_cast<const T*>(&r.q);
#pragma unroll
    for (int i = 0; i < VEC; ++i) out[i] = to_f(e[i]);
  }
}

template <typename T, int VEC, bool RES_BN>
__global__ void __launch_bounds__(kEwThreads, 3)
bn_apply_kernel(const T* __restrict__ x, const float* __restrict__ stats,
                const float* __restrict__ gamma, const float* __restrict__ beta,
                const T* __restrict__ res, const float* __restrict__ res_stats,
                const float* __restrict__ res_gamma, const float* __restrict__ res_beta,
                int relu, T* __restrict__ y, size_t nvec, int C, PartialSums ps) {
  __shared__ float s_stats[2 * 128];
  grid_dependency_wait();
  grid_dependency_release();
  const float* st = stats;
  if (ps.partial) { finalize_partials(ps, C, s_stats); st = s_stats; }
  const int cv = C / VEC;
  const size_t gtid = blockIdx.x * (size_t)blockDim.x + threadIdx.x, stride = (size_t)gridDim.x * blockDim.x;
  const int c0 = (int)(gtid % cv) * VEC;
  float mean[VEC], inv[VEC], ga[VEC], be[VEC], rmean[RES_BN ? VEC : 1], rinv[RES_BN ? VEC : 1], rga[RES_BN ? VEC : 1], rbe[RES_BN ? VEC : 1];
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    mean[j] = st[c0 + j]; inv[j] = st[C + c0 + j]; ga[j] = gamma[c0 + j]; be[j] = beta[c0 + j];
    if constexpr (RES_BN) { rmean[j] = res_stats[c0 + j]; rinv[j] = res_stats[C + c0 + j]; rga[j] = res_gamma[c0 + j]; rbe[j] = res_beta[c0 + j]; }
  }
  auto one = [&](size_t i, const RawVec<T, VEC>& xv, const RawVec<T, VEC>& rv) {
    float v[VEC], r[VEC], o[VEC];
    raw_to_f<T, VEC>(xv, v);
    if (res) raw_to_f<T, VEC>(rv, r);
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
      float t = ga[j] * ((v[j] - mean[j]) * inv[j]) + be[j];
      if (res) {
        float rr = r[j];
        if constexpr (RES_BN) rr = rga[j] * ((rr - rmean[j]) * rinv[j]) + rbe[j];
        t += rr;
      }
      o[j] = relu ? fmaxf(t, 0.f) : t;
    }
    store_vec<T, VEC>(y + i * VEC, o);
  };
  size_t i = gtid;
  for (; i + (kEwUnroll - 1) * stride < nvec; i += kEwUnroll * stride) {
    RawVec<T, VEC> xv[kEwUnroll], rv[kEwUnroll];
#pragma unroll
    for (int u = 0; u < kEwUnroll; ++u) xv[u] = load_raw<T, VEC>(x + (i + u * stride) * VEC);
    if (res) {
#pragma unroll
      for (int u = 0; u < kEwUnroll; ++u) rv[u] = load_raw<T, VEC>(res + (i + u * stride) * VEC);
    }
#pragma unroll
    for (int u = 0; u < kEwUnroll; ++u) one(i + u * stride, xv[u], rv[u]);
  }
  for (; i < nvec; i += stride) {
    RawVec<T, VEC> xv = load_raw<T, VEC>(x + i * VEC), rv = xv;
    if (res) rv = load_raw<T, VEC>(res + i * VEC);
    one(i, xv, rv);
  }
}

// ------------------------------------------------- batch norm, backward -----
// dz = dy * [mask > 0];  s0 = sum dz, s1 = sum dz*xhat (xhat from x, stats),
// s2 = sum dz*xhat2 (second normalised tensor sharing dz: the projection shortcut).
// The sums are the parameter gradients: dbeta = s0, dgamma = s1 (dgamma2 = s2, dbeta2 = s0).
template <typename T, int VEC, int NS>
__global__ void __launch_bounds__(kRedThreads)
bn_bwd_reduce_kernel(const T* __restrict__ dy, const T* __restrict__ mask, const T* __restrict__ x,
                     const float* __restrict__ stats, const T* __restrict__ x2, const float* __restrict__ stats2,
                     RedGeom g, float* __restrict__ sums, float* __restrict__ dgamma, float* __restrict__ dbeta,
                     float* __restrict__ dgamma2, float* __restrict__ dbeta2, float* __restrict__ partial,
                     unsigned int* __restrict__ counter) {
  const int C = g.ld;
  channel_reduce<NS, VEC>(
      g, partial, counter,
      [&](int row, int c0, float (&s)[NS][VEC]) {
        const size_t off = (size_t)row * C + c0;
        float d[VEC], m[VEC], v[VEC], v2[VEC];
        load_vec<T, VEC>(dy + off, d);
        if (mask) load_vec<T, VEC>(mask + off, m);
        load_vec<T, VEC>(x + off, v);
        if (NS == 3) load_vec<T, VEC>(x2 + off, v2);
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
          const int c = c0 + i;
          float dz = (mask && !(m[i] > 0.f)) ? 0.f : d[i];
          s[0][i] += dz;
          s[1][i] += dz * ((v[i] - stats[c]) * stats[C + c]);
          if (NS == 3) s[2][i] += dz * ((v2[i] - stats2[c]) * stats2[C + c]);
        }
      },
      [&](int c, double (&tot)[NS]) {
        sums[c] = (float)tot[0];
        sums[C + c] = (float)tot[1];
        dbeta[c] = (float)tot[0];
        dgamma[c] = (float)tot[1];
        if (NS == 3) {
          sums[2 * C + c] = (float)tot[2];
          dbeta2[c] = (float)tot[0];
          dgamma2[c] = (float)tot[2];
        }
      });
}

// dx = gamma*invstd*(dz - s0/M - xhat*s1/M) [+ res];  optionally the same for the second
// normalised tensor (dx2, TWO).  Per-thread channel constants and loads in flight as in bn_apply_kernel.
template <typename T, int VEC, bool TWO>
__global__ void __launch_bounds__(kEwThreads, 3)
bn_bwd_apply_kernel(const T* __restrict__ dy, const T* __restrict__ mask, const T* __restrict__ x,
                    const float* __restrict__ stats, const float* __restrict__ gamma,
                    const float* __restrict__ sums, const T* __restrict__ x2,
                    const float* __restrict__ stats2, const float* __restrict__ gamma2,
                    const T* __restrict__ res, T* __restrict__ dx, T* __restrict__ dx2,
                    size_t nvec, int C, float inv_m, PartialSums ps) {
  __shared__ float s_sums[2 * 128];
  grid_dependency_wait();
  grid_dependency_release();
  if (ps.partial) { finalize_partials(ps, C, s_sums); sums = s_sums; }
  const int cv = C / VEC;
  const size_t gtid = blockIdx.x * (size_t)blockDim.x + threadIdx.x, stride = (size_t)gridDim.x * blockDim.x;
  const int c0 = (int)(gtid % cv) * VEC;
  constexpr int V2 = TWO ? VEC : 1;
  float mean[VEC], inv[VEC], gi[VEC], s0[VEC], s1[VEC], mean2[V2], inv2[V2], gi2[V2], s2[V2];
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    mean[j] = stats[c0 + j]; inv[j] = stats[C + c0 + j]; gi[j] = gamma[c0 + j] * inv[j];
    s0[j] = sums[c0 + j] * inv_m; s1[j] = sums[C + c0 + j] * inv_m;
    if constexpr (TWO) { mean2[j] = stats2[c0 + j]; inv2[j] = stats2[C + c0 + j]; gi2[j] = gamma2[c0 + j] * inv2[j]; s2[j] = sums[2 * C + c0 + j] * inv_m; }
  }
  auto one = [&](size_t i, const RawVec<T, VEC>& dv, const RawVec<T, VEC>& mv, const RawVec<T, VEC>& xv) {
    float d[VEC], m[VEC], v[VEC], v2[VEC], r[VEC], o[VEC], o2[VEC];
    raw_to_f<T, VEC>(dv, d);
    if (mask) raw_to_f<T, VEC>(mv, m);
    raw_to_f<T, VEC>(xv, v);
    if constexpr (TWO) load_vec<T, VEC>(x2 + i * VEC, v2);
    if (res) load_vec<T, VEC>(res + i * VEC, r);
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
      const float dz = (mask && !(m[j] > 0.f)) ? 0.f : d[j];
      const float xh = (v[j] - mean[j]) * inv[j];
      const float t = gi[j] * (dz - s0[j] - xh * s1[j]);
      o[j] = res ? t + r[j] : t;
      if constexpr (TWO) {
        const float xh2 = (v2[j] - mean2[j]) * inv2[j];
        o2[j] = gi2[j] * (dz - s0[j] - xh2 * s2[j]);
      }
    }
    store_vec<T, VEC>(dx + i * VEC, o);
    if constexpr (TWO) store_vec<T, VEC>(dx2 + i * VEC, o2);
  };
  constexpr int U = 2;
  size_t i = gtid;
  for (; i + (U - 1) * stride < nvec; i += U * stride) {
    RawVec<T, VEC> dv[U], mv[U], xv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      dv[u] = load_raw<T, VEC>(dy + (i + u * stride) * VEC);
      mv[u] = mask ? load_raw<T, VEC>(mask + (i + u * stride) * VEC) : dv[u];
      xv[u] = load_raw<T, VEC>(x + (i + u * stride) * VEC);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) one(i + u * stride, dv[u], mv[u], xv[u]);
  }
  for (; i < nvec; i += stride) {
    RawVec<T, VEC> dv = load_raw<T, VEC>(dy + i * VEC), mv = dv, xv = load_raw<T, VEC>(x + i * VEC);
    if (mask) mv = load_raw<T, VEC>(mask + i * VEC);
    one(i, dv, mv, xv);
  }
}

// -------------------------------------------------------- small elementwise -
// out = scale * in  (the gradient-shrinking step, Eq. 15).
template <typename T, int VEC>
__global__ void scale_kernel(const T* __restrict__ in, T* __restrict__ out, float scale, size_t nvec) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < nvec; i += (size_t)gridDim.x * blockDim.x) {
    float v[VEC];
    load_vec<T, VEC>(in + i * VEC, v);
#pragma unroll
    for (int j = 0; j < VEC; ++j) v[j] *= scale;
    store_vec<T, VEC>(out + i * VEC, v);
  }
}

// out = a + b
template <typename T, int VEC>
__global__ void add_kernel(const T* __restrict__ a, const T* __restrict__ b, T* __restrict__ out, size_t nvec) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < nvec; i += (size_t)gridDim.x * blockDim.x) {
    float x[VEC], y[VEC];
    load_vec<T, VEC>(a + i * VEC, x);
    load_vec<T, VEC>(b + i * VEC, y);
#pragma unroll
    for (int j = 0; j < VEC; ++j) x[j] += y[j];
    store_vec<T, VEC>(out + i * VEC, x);
  }
}

// up[n][2p][2q][:] = dy[n][p][q][:], zero at the other pixels; dy [N][P][Q][C], up [N][2P][2Q][C], 16-byte vectors.
template <typename T, int VEC>
__global__ void upsample2_kernel(const T* __restrict__ dy, T* __restrict__ up, size_t nvec_up, int P, int Q, int C) {
  const int cv = C / VEC;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < nvec_up; i += (size_t)gridDim.x * blockDim.x) {
    const int c = (int)(i % cv);
    size_t pix = i / cv;
    const int w = (int)(pix % (2 * Q)); pix /= 2 * Q;
    const int h = (int)(pix % (2 * P));
    const size_t n = pix / (2 * P);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (((h | w) & 1) == 0) v = reinterpret_cast<const uint4*>(dy)[((n * P + (h >> 1)) * Q + (w >> 1)) * cv + c];
    reinterpret_cast<uint4*>(up)[i] = v;
  }
}

// Zero-padded shortcut of a block that changes the shape: out [N][P][Q][Co] = x [N][H][W][Ci] at every stride-th
// pixel, in channels lo .. lo+Ci-1 with lo = (Co - Ci)/2, zero elsewhere; and its backward, which puts the
// gated upstream gradient's middle channels back at those pixels of a zero [N][H][W][Ci] tensor.
template <typename T>
__global__ void pad_shortcut_kernel(const T* __restrict__ x, T* __restrict__ out, size_t rows_out, int P, int Q, int H, int W,
                                    int Ci, int Co, int stride) {
  const int lo = (Co - Ci) / 2;
  const size_t n = rows_out * (size_t)Co;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const int c = (int)(i % Co);
    size_t pix = i / Co;
    const int q = (int)(pix % Q); pix /= Q;
    const int p = (int)(pix % P);
    const size_t img = pix / P;
    T v = from_f<T>(0.f);
    if (c >= lo && c < lo + Ci) v = x[((img * H + (size_t)p * stride) * W + (size_t)q * stride) * Ci + (c - lo)];
    out[i] = v;
  }
}
template <typename T>
__global__ void pad_shortcut_bwd_kernel(const T* __restrict__ dy, const T* __restrict__ y, T* __restrict__ dx, size_t rows_in,
                                        int P, int Q, int H, int W, int Ci, int Co, int stride) {
  const int lo = (Co - Ci) / 2;
  const size_t n = rows_in * (size_t)Ci;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const int c = (int)(i % Ci);
    size_t pix = i / Ci;
    const int w = (int)(pix % W); pix /= W;
    const int h = (int)(pix % H);
    const size_t img = pix / H;
    T v = from_f<T>(0.f);
    if (h % stride == 0 && w % stride == 0) {
      const size_t o = ((img * P + h / stride) * Q + w / stride) * Co + lo + c;
      if (to_f(y[o]) > 0.f) v = dy[o];
    }
    dx[i] = v;
  }
}

// fp32 [rows][c_in] -> T [rows][c_out], channels c_in..c_out-1 zero (image ingest); labels copied alongside.
template <typename T>
__global__ void ingest_kernel(const float* __restrict__ img, T* __restrict__ out, size_t rows, int c_in, int c_out,
                              const int32_t* __restrict__ labels_in, int32_t* __restrict__ labels_out, int batch) {
  const size_t n = rows * (size_t)c_out;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const size_t row = i / c_out;
    const int c = (int)(i % c_out);
    out[i] = from_f<T>(c < c_in ? img[row * c_in + c] : 0.f);
  }
  if (blockIdx.x == 0)
    for (int i = threadIdx.x; i < batch; i += blockDim.x) labels_out[i] = labels_in[i];
}

// T [rows][c_src] -> fp32 [rows][c_dst] keeping the first c_dst channels (getters).
template <typename T>
__global__ void export_kernel(const T* __restrict__ in, float* __restrict__ out, size_t rows, int c_src, int c_dst) {
  const size_t n = rows * (size_t)c_dst;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const size_t row = i / c_dst;
    out[i] = to_f(in[row * c_src + (i % c_dst)]);
  }
}

// ------------------------------------------------------------------ head ----
// One block per sample: global average pool -> FC -> softmax cross-entropy, and the
// backward of all three down to the gradient of the pooled tensor's source.
//   x [B][HW][F] (T)   w [classes][F], b [classes] (fp32)
//   pooled [B][F], dlogits [B][classes], loss_n [B] (fp32 scratch for head_param_grad)
//   dx [B][HW][F] (T) = dpooled[f] / HW
// A label outside [0, classes) sets *bad_label and is treated as class 0.
// `groups` > 0 (F a multiple of the 16-byte vector, see head_groups): the sample is read and its gradient written in
// 16-byte vectors; `groups` sets of threads take every groups-th pixel and their partial sums are added in group
// order.  `groups` == 0: element by element, for any F.
template <typename T>
__global__ void head_fwd_bwd_kernel(const T* __restrict__ x, const float* __restrict__ w, const float* __restrict__ b,
                                    const int32_t* __restrict__ labels, int HW, int F, int classes, int batch, int groups,
                                    float* __restrict__ pooled, float* __restrict__ dlogits,
                                    float* __restrict__ loss_n, T* __restrict__ dx, int* __restrict__ bad_label) {
  constexpr int V = 16 / (int)sizeof(T);
  extern __shared__ __align__(16) float hs[];   // pooled[F] | dpooled[F] | partial[groups][F] | logits[classes]
  float* s_pool = hs;
  float* s_dpool = hs + F;
  float* s_part = s_dpool + F;
  float* s_logit = s_part + (size_t)groups * F;
  const int n = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
  const T* xn = x + (size_t)n * HW * F;
  if (groups > 0) {
    const int cols = F / V;
    for (int item = tid; item < groups * cols; item += nt) {
      const int g = item / cols, col = item - g * cols;
      float acc[V];
#pragma unroll
      for (int j = 0; j < V; ++j) acc[j] = 0.f;
#pragma unroll 4
      for (int p = g; p < HW; p += groups) {
        float v[V];
        load_vec<T, V>(xn + (size_t)p * F + col * V, v);
#pragma unroll
        for (int j = 0; j < V; ++j) acc[j] += v[j];
      }
#pragma unroll
      for (int j = 0; j < V; ++j) s_part[(size_t)g * F + col * V + j] = acc[j];
    }
    __syncthreads();
    for (int f = tid; f < F; f += nt) {
      float a = 0.f;
      for (int g = 0; g < groups; ++g) a += s_part[(size_t)g * F + f];
      a /= (float)HW;
      s_pool[f] = a;
      pooled[(size_t)n * F + f] = a;
    }
  } else {
    for (int f = tid; f < F; f += nt) {
      float a = 0.f;
#pragma unroll 8
      for (int p = 0; p < HW; ++p) a += to_f(xn[(size_t)p * F + f]);
      a /= (float)HW;
      s_pool[f] = a;
      pooled[(size_t)n * F + f] = a;
    }
  }
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31, nwarps = nt >> 5;
  for (int c = warp; c < classes; c += nwarps) {
    float a = 0.f;
    for (int f = lane; f < F; f += 32) a += w[(size_t)c * F + f] * s_pool[f];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if (lane == 0) s_logit[c] = a + b[c];
  }
  __syncthreads();
  __shared__ float s_max, s_sum;
  int label = labels[n];
  if (label < 0 || label >= classes) { if (tid == 0) atomicExch(bad_label, 1); label = 0; }
  if (warp == 0) {                       // the lanes share the classes; the partial sums meet in a fixed butterfly
    float m = -INFINITY;
    for (int c = lane; c < classes; c += 32) m = fmaxf(m, s_logit[c]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float s = 0.f;
    for (int c = lane; c < classes; c += 32) s += expf(s_logit[c] - m);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) {
      s_max = m; s_sum = s;
      loss_n[n] = -(s_logit[label] - m - logf(s));
    }
  }
  __syncthreads();
  for (int c = tid; c < classes; c += nt) {
    float p = expf(s_logit[c] - s_max) / s_sum;
    float d = (p - (c == label ? 1.f : 0.f)) / (float)batch;
    s_logit[c] = d;
    dlogits[(size_t)n * classes + c] = d;
  }
  __syncthreads();
  for (int f = tid; f < F; f += nt) {
    float a = 0.f;
#pragma unroll 4
    for (int c = 0; c < classes; ++c) a += w[(size_t)c * F + f] * s_logit[c];
    s_dpool[f] = a / (float)HW;
  }
  __syncthreads();
  T* dxn = dx + (size_t)n * HW * F;
  if (groups > 0) {
    // the row of F gradients, packed once as T into the (now free) partial-sum area, then copied to every pixel
    T* s_row = reinterpret_cast<T*>(s_part);
    for (int f = tid; f < F; f += nt) s_row[f] = from_f<T>(s_dpool[f]);
    __syncthreads();
    const int cols = F / V;
    const uint4* row4 = reinterpret_cast<const uint4*>(s_row);
    uint4* dx4 = reinterpret_cast<uint4*>(dxn);
    for (int i = tid; i < HW * cols; i += nt) dx4[i] = row4[i % cols];
  } else {
    for (int i = tid; i < HW * F; i += nt) dxn[i] = from_f<T>(s_dpool[i % F]);
  }
}

constexpr int kHeadThreads = 256;
// Pixel groups of head_fwd_bwd_kernel for F features of `elem_bytes` each: 0 when F is not a whole number of
// 16-byte vectors, otherwise as many as fill the block (at most 8, and within the default shared-memory limit).
inline int head_groups(int F, int classes, int HW, size_t elem_bytes) {
  const int V = (int)(16 / elem_bytes);
  if (F % V != 0) return 0;
  int g = kHeadThreads / (F / V);
  if (g > 8) g = 8;
  if (g > HW) g = HW;
  if (g < 1) g = 1;
  while (g > 1 && ((size_t)(2 + g) * F + classes) * 4 > 40 * 1024) --g;
  return g;
}
inline size_t head_smem_bytes(int F, int classes, int groups) { return ((size_t)(2 + groups) * F + classes) * 4; }

// dW[c][f] = sum_n dlogits[n][c]*pooled[n][f], db[c] = sum_n dlogits[n][c].  Grid (classes, ceil(F / 32)), 128
// threads: a lane owns a feature, the four warps take every fourth sample and their partial sums are added in warp
// order.  Blocks (c, 0) also form db[c]; block (0, 0) reduces the loss (mean over the batch) and raises *nonfinite if
// it is NaN/Inf.
__global__ void head_param_grad_kernel(const float* __restrict__ pooled, const float* __restrict__ dlogits,
                                       const float* __restrict__ loss_n, int F, int classes, int batch,
                                       float* __restrict__ dW, float* __restrict__ db, float* __restrict__ loss,
                                       int* __restrict__ nonfinite) {
  __shared__ float s_part[4][32];
  const int c = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int f = blockIdx.y * 32 + lane;
  float a = 0.f;
  if (f < F) {
#pragma unroll 8
    for (int n = warp; n < batch; n += 4) a += dlogits[(size_t)n * classes + c] * pooled[(size_t)n * F + f];
  }
  s_part[warp][lane] = a;
  __syncthreads();
  if (warp == 0 && f < F) dW[(size_t)c * F + f] = ((s_part[0][lane] + s_part[1][lane]) + s_part[2][lane]) + s_part[3][lane];
  if (blockIdx.y != 0) return;
  // the sums over the batch: lanes take every 32nd sample, the partial sums meet in a fixed butterfly
  if (warp == 1) {
    float s = 0.f;
    for (int n = lane; n < batch; n += 32) s += dlogits[(size_t)n * classes + c];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) db[c] = s;
  } else if (warp == 2 && c == 0) {
    double l = 0.0;
    for (int n = lane; n < batch; n += 32) l += (double)loss_n[n];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) {
      const float lf = (float)(l / (double)batch);
      *loss = lf;
      if (!isfinite(lf)) atomicExch(nonfinite, 1);
    }
  }
}

// The two launches of the head on stream `st` (arguments as the kernels').
template <typename T>
inline cudaError_t launch_head(cudaStream_t st, const T* x, const float* w, const float* b, const int32_t* labels, int HW,
                               int F, int classes, int batch, float* pooled, float* dlogits, float* loss_n, T* dx,
                               float* dW, float* db, float* loss, int* flags, bool second = true, bool first = true) {
  if (first) {
    int groups = head_groups(F, classes, HW, sizeof(T));
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(dx)) & 15) groups = 0;   // vectors need 16-byte alignment
    head_fwd_bwd_kernel<T><<<batch, kHeadThreads, head_smem_bytes(F, classes, groups), st>>>(
        x, w, b, labels, HW, F, classes, batch, groups, pooled, dlogits, loss_n, dx, flags + 1);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (second) {
    head_param_grad_kernel<<<dim3(classes, (F + 31) / 32), 128, 0, st>>>(pooled, dlogits, loss_n, F, classes, batch, dW, db,
                                                                          loss, flags);
    return cudaGetLastError();
  }
  return cudaSuccess;
}

// ------------------------------------------------------------------- SGD ----
// g' = g + wd*theta ; v = mu*v + g' ; theta -= lr*v   (v starts at 0, so the first
// update gives v = g').  Also writes the copies of theta the kernels compute with into
// the next weight-version slot: fp32 always, bf16 when next16 is given.  g is left untouched.
// The learning rate is `lr`, or *lr_dev when that pointer is given (a recorded launch can then
// follow a schedule without being re-recorded).
__global__ void sgd_kernel(float* __restrict__ theta, float* __restrict__ v, const float* __restrict__ g,
                           float* __restrict__ next32, __nv_bfloat16* __restrict__ next16, size_t n, float lr,
                           const float* __restrict__ lr_dev, float mu, float wd) {
  if (lr_dev) lr = *lr_dev;
  const size_t n4 = n / 4;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    float4 th = reinterpret_cast<float4*>(theta)[i];
    float4 vv = reinterpret_cast<float4*>(v)[i];
    const float4 gg = reinterpret_cast<const float4*>(g)[i];
    vv.x = mu * vv.x + (gg.x + wd * th.x); th.x -= lr * vv.x;
    vv.y = mu * vv.y + (gg.y + wd * th.y); th.y -= lr * vv.y;
    vv.z = mu * vv.z + (gg.z + wd * th.z); th.z -= lr * vv.z;
    vv.w = mu * vv.w + (gg.w + wd * th.w); th.w -= lr * vv.w;
    reinterpret_cast<float4*>(theta)[i] = th;
    reinterpret_cast<float4*>(v)[i] = vv;
    reinterpret_cast<float4*>(next32)[i] = th;
    if (next16) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(th.x, th.y), hi = __floats2bfloat162_rn(th.z, th.w);
      uint2 pk;
      pk.x = *reinterpret_cast<unsigned int*>(&lo);
      pk.y = *reinterpret_cast<unsigned int*>(&hi);
      reinterpret_cast<uint2*>(next16)[i] = pk;
    }
  }
  if (blockIdx.x == 0)
    for (size_t i = n4 * 4 + threadIdx.x; i < n; i += blockDim.x) {
      float vv = mu * v[i] + (g[i] + wd * theta[i]);
      float th = theta[i] - lr * vv;
      v[i] = vv; theta[i] = th;
      next32[i] = th;
      if (next16) next16[i] = __float2bfloat16_rn(th);
    }
}

__global__ void set_scalar_kernel(float* dst, float value) { *dst = value; }

// fp32 -> T copy (refreshing the compute copies after fdg_set_params).
template <typename T>
__global__ void cast_kernel(const float* __restrict__ in, T* __restrict__ out, size_t n) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    out[i] = from_f<T>(in[i]);
}

// ------------------------------------------------------------- inference ----
// Inference-mode statistics of all batch norms of a module in one launch: for table entry e,
// out[soff .. soff+C) = running mean, out[soff+C .. soff+2C) = 1/sqrt(running variance + eps).
struct EvalStatEntry { size_t roff, soff; int C; };
__global__ void bn_eval_stats_kernel(const float* __restrict__ running, float* __restrict__ out,
                                     const EvalStatEntry* __restrict__ table, float eps) {
  const EvalStatEntry e = table[blockIdx.x];
  for (int c = threadIdx.x; c < e.C; c += blockDim.x) {
    out[e.soff + c] = running[e.roff + c];
    out[e.soff + e.C + c] = 1.f / sqrtf(running[e.roff + e.C + c] + eps);
  }
}

// Classifier in inference mode, one block per sample: global average pool -> FC -> logits (optional copy
// out) -> arg-max (lowest index among equal logits) compared with the label; *correct counts the matches.
template <typename T>
__global__ void head_eval_kernel(const T* __restrict__ x, const float* __restrict__ w, const float* __restrict__ b,
                                 const int32_t* __restrict__ labels, int HW, int F, int classes,
                                 float* __restrict__ logits_out, int* __restrict__ correct) {
  extern __shared__ float hs[];            // pooled[F] | logits[classes]
  float* s_pool = hs;
  float* s_logit = hs + F;
  const int n = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
  const T* xn = x + (size_t)n * HW * F;
  for (int f = tid; f < F; f += nt) {
    float a = 0.f;
    for (int p = 0; p < HW; ++p) a += to_f(xn[(size_t)p * F + f]);
    s_pool[f] = a / (float)HW;
  }
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31, nwarps = nt >> 5;
  for (int c = warp; c < classes; c += nwarps) {
    float a = 0.f;
    for (int f = lane; f < F; f += 32) a += w[(size_t)c * F + f] * s_pool[f];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if (lane == 0) { s_logit[c] = a + b[c]; if (logits_out) logits_out[(size_t)n * classes + c] = a + b[c]; }
  }
  __syncthreads();
  if (tid == 0 && labels && correct) {
    int best = 0;
    for (int c = 1; c < classes; ++c) if (s_logit[c] > s_logit[best]) best = c;
    if (best == labels[n]) atomicAdd(correct, 1);
  }
}

// ---------------------------------------------------------- host launchers ---
// Shared by the module runtime and the operator-level entry points, so that both issue the same
// kernels in the same launch shapes.
inline int ew_blocks(size_t nvec) {
  size_t b = (nvec + 255) / 256;
  return (int)(b < 1 ? 1 : (b > 148 * 8 ? 148 * 8 : b));
}
template <typename T> constexpr int full_vec() { return 16 / sizeof(T); }

// Floats of scratch a channel reduction over C channels may write (per-block partial sums).
inline size_t red_scratch_floats(int C) { return (size_t)kRedMaxBlocks * kRedMaxSums * C; }

// stats[0..C) = mean, stats[C..2C) = 1/sqrt(var + eps) of x [rows][C]; `counter` is a zeroed ticket word
// (the kernel leaves it zero again).
template <typename T>
inline cudaError_t launch_bn_stats(cudaStream_t st, const T* x, size_t rows, int C, float eps, float* stats,
                                   float* scratch, unsigned int* counter, float* running = nullptr, float momentum = 0.f) {
  constexpr int V = full_vec<T>();
  const RunningStats run{running, momentum, rows > 1 ? (float)((double)rows / (double)(rows - 1)) : 1.f};
  if (C % V == 0) {
    RedGeom g = red_geom((int)rows, C, V);
    bn_stats_kernel<T, V><<<dim3(g.blocks, g.slabs), kRedThreads, (size_t)(g.rp > 2 ? g.rp : 2) * 2 * g.C * 4, st>>>(x, g, eps, stats, scratch, counter, run);
  } else {
    RedGeom g = red_geom((int)rows, C, 1);
    bn_stats_kernel<T, 1><<<dim3(g.blocks, g.slabs), kRedThreads, (size_t)(g.rp > 2 ? g.rp : 2) * 2 * g.C * 4, st>>>(x, g, eps, stats, scratch, counter, run);
  }
  return cudaGetLastError();
}

// Grid of the batch-norm apply kernels: what `nvec` vectors need, bounded by `cap` (0 = none), and such that
// the grid's thread count is a multiple of the `cv` channel vectors of a row (every thread then stays on the
// same channels).  Surplus blocks of a tiny tensor simply find no work.
inline int ew_grid_for_channels(size_t nvec, int cv, int cap) {
  int a = cv, b = kEwThreads;
  while (b) { const int t = a % b; a = b; b = t; }
  const int unit = cv / a;                       // blocks per period
  int blocks = ew_blocks((nvec + kEwUnroll - 1) / kEwUnroll);
  if (cap > 0 && blocks > cap) blocks = cap;
  blocks = blocks / unit * unit;
  return blocks < unit ? unit : blocks;
}

// y = [relu](BN(x) + residual).  `partial` != null: the statistics are not in `stats` yet; a convolution left
// `nparts` rows of per-CTA sums (sum x, sum x^2) there, which every block adds up first (block 0 saves the
// result to `stats`); `block_cap` then bounds the grid, since every block repeats that addition.
template <typename T>
inline cudaError_t launch_bn_apply(cudaStream_t st, const T* x, float* stats, const float* gamma, const float* beta,
                                   const T* res, const float* res_stats, const float* res_gamma, const float* res_beta,
                                   bool relu, T* y, size_t rows, int C, float eps, const float* partial, int nparts,
                                   int block_cap, float* running = nullptr, float momentum = 0.f) {
  constexpr int V = full_vec<T>();
  const size_t n = rows * C;
  PartialSums ps{};
  if (partial && nparts > 0) {
    if (2 * C > kEwThreads) return cudaErrorInvalidValue;
    ps.partial = partial; ps.nparts = nparts; ps.kind = 1; ps.inv_count = 1.f / (float)rows; ps.eps = eps;
    ps.save0 = stats; ps.save1 = stats + C;
    ps.run = RunningStats{running, momentum, rows > 1 ? (float)((double)rows / (double)(rows - 1)) : 1.f};
  }
  if (C % V == 0) {
    const int blocks = ew_grid_for_channels(n / V, C / V, ps.partial ? block_cap : 0);
    if (res_stats) return launch_chained(bn_apply_kernel<T, V, true>, blocks, kEwThreads, 0, st, x, stats, gamma, beta, res, res_stats, res_gamma, res_beta, (int)relu, y, n / V, C, ps);
    return launch_chained(bn_apply_kernel<T, V, false>, blocks, kEwThreads, 0, st, x, stats, gamma, beta, res, res_stats, res_gamma, res_beta, (int)relu, y, n / V, C, ps);
  }
  const int blocks = ew_grid_for_channels(n, C, 0);
  if (res_stats) return launch_chained(bn_apply_kernel<T, 1, true>, blocks, kEwThreads, 0, st, x, stats, gamma, beta, res, res_stats, res_gamma, res_beta, (int)relu, y, n, C, ps);
  return launch_chained(bn_apply_kernel<T, 1, false>, blocks, kEwThreads, 0, st, x, stats, gamma, beta, res, res_stats, res_gamma, res_beta, (int)relu, y, n, C, ps);
}

// First half of the batch-norm backward: the per-channel sums of dz = dy*[mask>0] (and dz*xhat, dz*xhat2),
// which are also the parameter gradients; totals to `sums` [3*C].
template <typename T>
inline cudaError_t launch_bn_bwd_reduce(cudaStream_t st, const T* dy, const T* mask, const T* x, const float* stats,
                                        const T* x2, const float* stats2, size_t rows, int C, float* sums,
                                        float* dgamma, float* dbeta, float* dgamma2, float* dbeta2, float* scratch,
                                        unsigned int* counter) {
  constexpr int V = full_vec<T>();
  const bool two = x2 != nullptr, vec = C % V == 0;
  const int ns = two ? 3 : 2;
  RedGeom g = red_geom((int)rows, C, vec ? V : 1);
  const size_t smem = (size_t)(g.rp > 2 ? g.rp : 2) * ns * g.C * 4;
#define FDG_RED(VV, NS) bn_bwd_reduce_kernel<T, VV, NS><<<dim3(g.blocks, g.slabs), kRedThreads, smem, st>>>( \
      dy, mask, x, stats, x2, stats2, g, sums, dgamma, dbeta, dgamma2, dbeta2, scratch, counter)
  if (vec) { if (two) FDG_RED(V, 3); else FDG_RED(V, 2); }
  else     { if (two) FDG_RED(1, 3); else FDG_RED(1, 2); }
#undef FDG_RED
  return cudaGetLastError();
}

// Second half: dx = gamma*invstd*(dz - s0/M - xhat*s1/M) [+ res] (and dx2 for the second normalised tensor).
// The sums come from `sums`, or, when `partial` != null, from `nparts` rows of per-CTA sums (sum dz, sum dz*xhat)
// left by the data-gradient kernel that produced dy (block 0 then also writes dbeta / dgamma).
template <typename T>
inline cudaError_t launch_bn_bwd_apply(cudaStream_t st, const T* dy, const T* mask, const T* x, const float* stats,
                                       const float* gamma, const float* sums, const T* x2, const float* stats2,
                                       const float* gamma2, const T* res, T* dx, T* dx2, size_t rows, int C,
                                       const float* partial, int nparts, float* dgamma, float* dbeta, int block_cap) {
  constexpr int V = full_vec<T>();
  const size_t n = rows * C;
  const float inv_m = 1.f / (float)rows;
  PartialSums ps{};
  if (partial && nparts > 0) {
    if (2 * C > kEwThreads) return cudaErrorInvalidValue;
    ps.partial = partial; ps.nparts = nparts; ps.kind = 2; ps.save0 = dbeta; ps.save1 = dgamma;
  }
  if (C % V == 0) {
    const int blocks = ew_grid_for_channels(n / V, C / V, ps.partial ? block_cap : 0);
    if (dx2) return launch_chained(bn_bwd_apply_kernel<T, V, true>, blocks, kEwThreads, 0, st, dy, mask, x, stats, gamma, sums, x2, stats2, gamma2, res, dx, dx2, n / V, C, inv_m, ps);
    return launch_chained(bn_bwd_apply_kernel<T, V, false>, blocks, kEwThreads, 0, st, dy, mask, x, stats, gamma, sums, x2, stats2, gamma2, res, dx, dx2, n / V, C, inv_m, ps);
  }
  const int blocks = ew_grid_for_channels(n, C, 0);
  if (dx2) return launch_chained(bn_bwd_apply_kernel<T, 1, true>, blocks, kEwThreads, 0, st, dy, mask, x, stats, gamma, sums, x2, stats2, gamma2, res, dx, dx2, n, C, inv_m, ps);
  return launch_chained(bn_bwd_apply_kernel<T, 1, false>, blocks, kEwThreads, 0, st, dy, mask, x, stats, gamma, sums, x2, stats2, gamma2, res, dx, dx2, n, C, inv_m, ps);
}

template <typename T>
inline cudaError_t launch_scale(cudaStream_t st, const T* in, T* out, float s, size_t n) {
  constexpr int V = full_vec<T>();
  if (n % V == 0) scale_kernel<T, V><<<ew_blocks(n / V), 256, 0, st>>>(in, out, s, n / V);
  else scale_kernel<T, 1><<<ew_blocks(n), 256, 0, st>>>(in, out, s, n);
  return cudaGetLastError();
}

inline cudaError_t launch_sgd(cudaStream_t st, float* theta, float* v, const float* g, float* next32,
                              __nv_bfloat16* next16, size_t n, float lr, const float* lr_dev, float mu, float wd) {
  size_t b = (n / 4 + 255) / 256;
  const int blocks = (int)(b < 1 ? 1 : (b > 148 * 8 ? 148 * 8 : b));
  sgd_kernel<<<blocks, 256, 0, st>>>(theta, v, g, next32, next16, n, lr, lr_dev, mu, wd);
  return cudaGetLastError();
}

template <typename T>
inline cudaError_t launch_ingest(cudaStream_t st, const float* img, T* out, size_t rows, int c_in, int c_out,
                                 const int32_t* labels_in, int32_t* labels_out, int batch) {
  ingest_kernel<T><<<ew_blocks(rows * c_out), 256, 0, st>>>(img, out, rows, c_in, c_out, labels_in, labels_out, batch);
  return cudaGetLastError();
}

}  // namespace fdg
