// libfdg: the module runtime and the C ABI (see include/fdg.h for the contract).
//
// One context holds K modules.  Each module owns, inside the caller's workspace:
//   * fp32 master parameters, momentum and the last gradient (flat vectors);
//   * a ring of weight versions: the copy of the parameters the kernels compute with,
//     written by the update kernel, so that the delayed backward of a batch can read
//     the weights its forward used (superscripts of Eq. 10);
//   * an activation FIFO: one slot per batch in flight holding everything the backward
//     of that batch needs (what Fig. 1(b) keeps as the computation graph saved by the forward);
//   * a gradient mailbox (ring of 3) that receives the gradient of the module input
//     and is read by the upstream module in the next iteration (Section 3.1,
//     "communication");
//   * private temporaries.
// A module reads its input straight from the upstream module's FIFO slot, so the
// "send" of an activation is the producer's own store and the "receive" is a stream
// event.  Nothing is copied between modules.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <climits>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/fdg.h"
#include "../../include/fdg_ops.h"
#include "conv_dispatch.cuh"
#include "elementwise.cuh"

namespace fdg {

typedef __nv_bfloat16 bf16;
constexpr int kEventRing = 4;
constexpr size_t kLogIterations = 4096;
constexpr int kRedPartialCtas = 256;                 // upper bound of the CTAs of one convolution launch
constexpr float kBnMomentum = 0.1f;                  // weight of the newest batch in the running statistics

enum UnitType { U_STEM, U_BASIC, U_PREACT, U_HEAD };

// Kernel classes for the optional per-launch profiler (fdg_profile_enable).
enum KClass { KC_CONV_FPROP, KC_CONV_DGRAD, KC_CONV_WGRAD, KC_BN_STATS, KC_BN_APPLY, KC_BN_BWD_REDUCE,
              KC_BN_BWD_APPLY, KC_HEAD, KC_SGD, KC_SHRINK, KC_INGEST, KC_COUNT };
static const char* const kClassNames[KC_COUNT] = {"conv_fprop", "conv_dgrad", "conv_wgrad", "bn_stats", "bn_apply",
                                                  "bn_bwd_reduce", "bn_bwd_apply", "head", "sgd", "shrink", "ingest"};
constexpr size_t kProfMaxPairs = 1 << 16;
struct ProfRec { int cls; double bytes, flops; };

// One gradient tensor of a module's backward pass that fdg_capture_begin can keep a copy of.
struct CaptureEntry { int unit, which, ch; size_t off, elems; };

struct Unit {
  UnitType type;
  int index;                 // 0 stem, b block, -1 head
  int ci, co, stride;
  bool proj;
  bool zpad;                 // shape change bridged by the parameter-free zero-padded shortcut
  bool bn;                   // stem: has BN+ReLU (6n+2); head: has BN+ReLU (WRN)
  int H, W, P, Q;            // input / output spatial size
  // offsets into the module's flat parameter vector
  size_t w1, g1, b1, w2, g2, b2, ws, gs, bs;
  // offsets (elements of T) of saved tensors inside an activation-FIFO slot; y is the unit output
  size_t t_a, t_b, t_c, t_y, t_s;
  // offsets (floats) of saved statistics inside the slot's fp32 region
  size_t st1, st2, sts;
  // offsets of the flipped copies of w1 / w2 (and of the transposed 1x1 shortcut filter) inside a wflip16 slot, or -1
  // when that conv's dgrad is not on tensor cores
  long long f1 = -1, f2 = -1, fs = -1;
  // offsets of the running statistics (mean[C], var[C]) of BN1 / BN2 / the shortcut BN in the module's vector, or -1
  long long r1 = -1, r2 = -1, rs = -1;
};

struct Module {
  int k;                                   // 1-based
  std::vector<Unit> units;
  std::vector<fdg_param_entry> layout;
  size_t n_params = 0;
  int D = 1;                               // activation-FIFO depth
  int Dw = 1;                              // weight versions kept
  int Din = 0;                             // image ring depth (module 1 only)
  size_t slot_elems = 0, slot_floats = 0;  // per FIFO slot
  size_t in_elems = 0, out_elems = 0;      // module input / output tensor sizes (stored channels)
  int in_h = 0, in_w = 0, in_c = 0, in_c_logical = 0, out_c = 0;
  size_t max_act = 0;                      // largest activation tensor (elements)
  size_t scratch_floats = 0;               // reduction partials / weight-gradient slices
  // device pointers
  float *theta = nullptr, *mom = nullptr, *grad = nullptr, *wver = nullptr;
  bf16* wver16 = nullptr;
  bf16* wflip16 = nullptr;                 // Dw copies of the flipped/transposed 3x3 weights (dgrad operands)
  size_t flip_elems = 0;
  unsigned flip_blocks = 8;                // blocks per table entry of the flip kernel: one per 8192 weights of the largest
  std::vector<tc::FlipEntry> flip_table;   // host copy; src = offset in a wver16 slot, dst = offset in a wflip16 slot
  tc::FlipEntry* flip_table_dev = nullptr;
  char* fifo = nullptr;                    // D slots of slot_elems*sizeof(T)
  float* fifo_f = nullptr;                 // D slots of slot_floats
  char* in_ring = nullptr;                 // module 1: Din image slots
  char* mail = nullptr;                    // kMailRing slots of in_elems (k >= 2)
  char* temps[6] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
  float *scratch = nullptr, *bnsums = nullptr;
  float* wscratch = nullptr;               // partial sums of the weight-gradient kernels (they run on the side stream)
  size_t wscratch_floats = 0;
  unsigned int* counter = nullptr;
  char* up = nullptr;                      // dy of a stride-2 convolution spread onto the input's pixel grid
  size_t up_elems = 0;
  float* red_partial = nullptr;            // per-CTA partial sums of the reductions fused into convolution epilogues
  size_t red_partial_floats = 0;
  unsigned int* red_counter = nullptr;
  float *pooled = nullptr, *dlogits = nullptr, *loss_n = nullptr, *loss = nullptr;   // head
  // host state
  int64_t updates = 0;
  std::vector<int64_t> slot_version, slot_batch;
  int64_t last_out_batch = -1, last_grad_batch = -1;
  int last_out_slot = -1, last_grad_slot = -1;
  cudaStream_t stream = nullptr;
  cudaStream_t stream2 = nullptr;          // side stream: weight gradients run beside the data-gradient chain
  cudaEvent_t ev_fork2 = nullptr, ev_join2 = nullptr, ev_buf[4] = {nullptr, nullptr, nullptr, nullptr};
  cudaEvent_t ev_act[kEventRing], ev_grad[kEventRing];
  // running batch-norm statistics (inference): flat vector, and the table the inference pass reads them through
  float* running = nullptr;
  size_t n_running = 0;
  std::vector<EvalStatEntry> eval_table;
  EvalStatEntry* eval_table_dev = nullptr;
  // gradient capture (fdg_capture_begin): where each gradient tensor of a backward pass is copied to
  std::vector<CaptureEntry> cap_table;
  size_t cap_elems = 0;
  char* cap_buf = nullptr;
  int64_t cap_batch = -1;
};

}  // namespace fdg

using namespace fdg;

struct fdg_ctx {
  fdg_arch arch;
  fdg_config cfg;
  std::vector<int> splits;
  int K = 0;
  bool bf16_mode = false;
  size_t esize = 4;
  std::vector<Module> mods;
  bool own_streams = false;
  cudaEvent_t ev_in[kEventRing];
  cudaEvent_t ev_join;
  int32_t* labels = nullptr;          // ring of label_ring batches
  int label_ring = 0;
  int* flags = nullptr;               // [0] non-finite loss, [1] label out of range, [2] a tensor-core kernel's wait ran out,
                                      // [3] result word of the guard check
  std::vector<size_t> guard_offsets;  // byte offsets of the guard regions behind the workspace buffers
  unsigned long long* guard_table = nullptr;   // the same on the device
  float* staging = nullptr;           // fp32 staging for getters
  float* host_images = nullptr;       // device staging of fdg_step_host
  int32_t* host_labels = nullptr;
  size_t staging_elems = 0;
  int64_t t = 0;
  int64_t last_batch = INT64_MAX;     // no batch beyond this one exists (set while draining)
  bool has_schedule = false;
  fdg_lr_schedule schedule;
  char* ws_base = nullptr;            // the caller's workspace, as carved
  size_t ws_bytes = 0;
  float lr = 0.f;
  uint64_t launches = 0;
  std::vector<fdg_sched_entry> log;
  mutable std::string err;
  fdg_status latched = FDG_OK;
  int device = 0;
  fdg::TensorMapCache tmaps;
  // ring sizes that do not depend on the module
  int mail_ring = 3;
  // CUDA-graph replay (cfg.graphs): one executable graph per phase of the rings
  bool use_graphs = false;
  int period = 1;                     // all ring sizes divide it
  int ew_block_cap = 2 * 148;         // grid bound of the batch-norm apply kernels that re-add partial sums
  bool graph_mode_entered = false;
  std::vector<cudaGraphExec_t> graph_exec;
  std::vector<uint64_t> graph_sig, graph_launches;
  uint64_t step_sig = 0;              // signature of the slots the current iteration touches
  cudaStream_t cap_stream = nullptr;  // origin stream of the recordings (the caller's stream may be the legacy
                                      // default stream, which cannot be captured); graphs are launched on the caller's
  cudaEvent_t ev_fork = nullptr;
  // fdg_step_host: the host-to-device copy of a call runs on its own stream, beside the step of the call before;
  // ev_staged = the copy has landed, ev_ingested = the ingest kernel has read the staging buffers (they may be refilled)
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_staged = nullptr, ev_ingested = nullptr;
  bool record_ingested = false;
  std::vector<cudaEvent_t> ev_cjoin;
  float* lr_dev = nullptr;
  float lr_on_device = -1.f;
  int* tc_error = nullptr;            // device word raised by a tensor-core kernel whose wait timed out
  cudaStream_t last_stream = nullptr;   // stream of the most recent fdg_step
  bool stepped = false;
  // profiler
  bool profiling = false;
  std::vector<cudaEvent_t> prof_events;     // 2 per recorded launch
  std::vector<fdg::ProfRec> prof_recs;
  std::vector<cudaEvent_t> mod_events;      // 2 per recorded module pass (forward, or backward + update)
  std::vector<int> mod_event_owner;         // module (0-based) of each pair
};

namespace fdg {

// ------------------------------------------------------------------ planning --
static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Every buffer carved out of the workspace is followed by kGuardBytes that no kernel may write: they are
// filled with a pattern at creation and compared on request (fdg_debug_check_guards), so a kernel that
// runs past the end of its buffer is found at the buffer it overran instead of in its neighbour's results.
constexpr size_t kGuardBytes = 256;
constexpr unsigned int kGuardWord = 0xA5C3F00Du;
struct Carver {
  char* base;
  size_t off = 0;
  size_t count = 0;                        // buffers taken so far
  std::vector<size_t>* guards = nullptr;   // byte offsets of the guard regions, in order (recorded when set)
  explicit Carver(char* b) : base(b) {}
  template <typename P> P* take(size_t bytes) {
    off = align_up(off, 256);
    P* p = base ? reinterpret_cast<P*>(base + off) : nullptr;
    off = align_up(off + bytes, 256);
    if (guards) guards->push_back(off);
    off += kGuardBytes;
    ++count;
    return p;
  }
};
__global__ void guard_fill_kernel(char* __restrict__ base, const unsigned long long* __restrict__ offsets) {
  reinterpret_cast<unsigned int*>(base + offsets[blockIdx.x])[threadIdx.x] = kGuardWord;
}
// *first_bad = the lowest index of a guard region that no longer holds the pattern (left untouched if all do)
__global__ void guard_check_kernel(const char* __restrict__ base, const unsigned long long* __restrict__ offsets,
                                   int* __restrict__ first_bad) {
  if (reinterpret_cast<const unsigned int*>(base + offsets[blockIdx.x])[threadIdx.x] != kGuardWord)
    atomicMin(first_bad, (int)blockIdx.x);
}

static int conv_out(int n, int r, int stride, int pad) { return (n + 2 * pad - r) / stride + 1; }
static int pow2_at_least(int x) { int p = 1; while (p < x) p <<= 1; return p; }

static fdg_status validate(const fdg_arch* a, const fdg_config* c, std::string* why) {
  if (!a || !c) { *why = "null arch or config"; return FDG_ERR_INVALID_ARG; }
  if (a->family != FDG_RESNET_6N2 && a->family != FDG_WRN) { *why = "unknown family"; return FDG_ERR_INVALID_ARG; }
  if (a->n_stages < 1 || a->n_stages > 4 || a->stem_width < 1 || a->in_h < 4 || a->in_w < 4 || a->in_c < 1 || a->num_classes < 2 ||
      a->batch < 1 || !(a->bn_eps > 0.f)) { *why = "bad architecture sizes"; return FDG_ERR_INVALID_ARG; }
  for (int i = 0; i < a->n_stages; ++i) if (a->widths[i] < 1 || a->blocks[i] < 1) { *why = "bad stage width or block count"; return FDG_ERR_INVALID_ARG; }
  const int down = 1 << (a->n_stages - 1);
  if (a->in_h % down || a->in_w % down) { *why = "image size must be a multiple of 2^(stages-1)"; return FDG_ERR_INVALID_ARG; }
  if (a->shortcut != FDG_SHORTCUT_PROJECTION && a->shortcut != FDG_SHORTCUT_ZERO_PAD) { *why = "unknown shortcut"; return FDG_ERR_INVALID_ARG; }
  if (a->shortcut == FDG_SHORTCUT_ZERO_PAD) {
    if (a->family != FDG_RESNET_6N2) { *why = "the zero-padded shortcut belongs to the post-activation family"; return FDG_ERR_INVALID_ARG; }
    int prev = a->stem_width;
    for (int i = 0; i < a->n_stages; ++i) {
      if (a->widths[i] < prev || (a->widths[i] - prev) % 2) { *why = "zero-padded shortcut needs widths that grow by an even amount"; return FDG_ERR_INVALID_ARG; }
      prev = a->widths[i];
    }
  }
  if (c->K < 1 || c->K > 64) { *why = "K out of range"; return FDG_ERR_INVALID_ARG; }
  if (c->K > 1 && !c->split_after_block) { *why = "split_after_block is null"; return FDG_ERR_INVALID_ARG; }
  int nblocks = 0;
  for (int i = 0; i < a->n_stages; ++i) nblocks += a->blocks[i];
  int prev = 0;
  for (int i = 0; i + 1 < c->K; ++i) {
    int s = c->split_after_block[i];
    if (s <= prev || s >= nblocks) { *why = "split points must ascend inside [1, blocks-1]"; return FDG_ERR_INVALID_ARG; }
    prev = s;
  }
  if (!(c->beta > 0.f && c->beta <= 1.f)) { *why = "beta must be in (0, 1]"; return FDG_ERR_INVALID_ARG; }
  if (!(c->lr >= 0.f) || !(c->momentum >= 0.f && c->momentum < 1.f) || !(c->weight_decay >= 0.f)) {
    *why = "bad optimiser constants"; return FDG_ERR_INVALID_ARG; }
  if ((c->order != FDG_BACKWARD_FIRST && c->order != FDG_FORWARD_FIRST) ||
      (c->weight_reading != FDG_STASHED && c->weight_reading != FDG_CURRENT) ||
      (c->precision != FDG_FP32_CUDACORE && c->precision != FDG_BF16_TC)) { *why = "bad enum value"; return FDG_ERR_INVALID_ARG; }
  // channel counts the vectorised kernels can address
  const int vec = c->precision == FDG_BF16_TC ? 8 : 4;
  int chans[5] = {a->stem_width, a->widths[0], a->widths[0], a->widths[0], a->widths[0]};
  for (int i = 0; i < a->n_stages; ++i) chans[1 + i] = a->widths[i];
  for (int ch : chans) {
    if ((ch % vec != 0 && ch > kRedThreads) || ch / vec > kRedThreads) { *why = "channel count not addressable by the reduction kernels"; return FDG_ERR_UNSUPPORTED; }
    if (c->precision == FDG_BF16_TC && ch % 8 != 0) { *why = "bf16 mode needs channel counts that are multiples of 8"; return FDG_ERR_UNSUPPORTED; }
  }
  if ((size_t)a->batch * a->in_h * a->in_w * (size_t)std::max({chans[0], chans[1], chans[2], chans[3], chans[4]}) > (size_t)1 << 31) {
    *why = "activation tensor exceeds 2^31 elements"; return FDG_ERR_UNSUPPORTED; }
  return FDG_OK;
}

static void add_param(Module& m, int kind, int unit, int d0, int d1, int d2, int d3, size_t* off_out) {
  fdg_param_entry e;
  e.kind = kind; e.unit = unit; e.dims[0] = d0; e.dims[1] = d1; e.dims[2] = d2; e.dims[3] = d3;
  e.offset = m.n_params; e.count = (size_t)d0 * d1 * d2 * d3;
  *off_out = e.offset;
  m.n_params += e.count;
  m.layout.push_back(e);
}

static long long add_running(Module& m, int C) {
  const long long off = (long long)m.n_running;
  m.n_running += (size_t)2 * C;
  return off;
}

// Builds the unit lists, parameter tables and slot layouts of all modules (no pointers yet).
static void plan_modules(fdg_ctx* c) {
  const fdg_arch& a = c->arch;
  const int K = c->K;
  const bool wrn = a.family == FDG_WRN;
  int nblocks = 0;
  for (int i = 0; i < a.n_stages; ++i) nblocks += a.blocks[i];
  c->mods.assign(K, Module());
  std::vector<int> last_block(K);
  for (int k = 0; k < K; ++k) last_block[k] = (k + 1 < K) ? c->splits[k] : nblocks;

  int k = 0;
  int H = a.in_h, W = a.in_w, ci = a.stem_width;
  const int in_c_store = a.in_c;
  for (int kk = 0; kk < K; ++kk) c->mods[kk].k = kk + 1;
  {   // stem
    Module& m = c->mods[0];
    Unit u{}; u.type = U_STEM; u.index = 0; u.ci = in_c_store; u.co = a.stem_width; u.stride = 1; u.bn = !wrn;
    u.H = H; u.W = W; u.P = H; u.Q = W;
    add_param(m, FDG_PARAM_CONV, 0, u.co, 3, 3, a.in_c, &u.w1);
    if (u.bn) { add_param(m, FDG_PARAM_BN_GAMMA, 0, u.co, 1, 1, 1, &u.g1); add_param(m, FDG_PARAM_BN_BETA, 0, u.co, 1, 1, 1, &u.b1); u.r1 = add_running(m, u.co); }
    m.units.push_back(u);
    m.in_h = H; m.in_w = W; m.in_c = in_c_store; m.in_c_logical = a.in_c;
  }
  for (int b = 1; b <= nblocks; ++b) {
    while (b > last_block[k]) ++k;
    Module& m = c->mods[k];
    int stage = 0, j = b - 1;
    while (j >= a.blocks[stage]) { j -= a.blocks[stage]; ++stage; }
    Unit u{}; u.type = wrn ? U_PREACT : U_BASIC; u.index = b; u.ci = ci; u.co = a.widths[stage];
    u.stride = (stage > 0 && j == 0) ? 2 : 1;
    const bool changes = (u.ci != u.co) || u.stride != 1;
    u.proj = changes && a.shortcut == FDG_SHORTCUT_PROJECTION;
    u.zpad = changes && a.shortcut == FDG_SHORTCUT_ZERO_PAD;
    u.H = H; u.W = W; u.P = conv_out(H, 3, u.stride, 1); u.Q = conv_out(W, 3, u.stride, 1);
    if (m.units.empty()) { m.in_h = H; m.in_w = W; m.in_c = ci; m.in_c_logical = ci; }
    if (!wrn) {
      add_param(m, FDG_PARAM_CONV, b, u.co, 3, 3, u.ci, &u.w1);
      add_param(m, FDG_PARAM_BN_GAMMA, b, u.co, 1, 1, 1, &u.g1); add_param(m, FDG_PARAM_BN_BETA, b, u.co, 1, 1, 1, &u.b1);
      add_param(m, FDG_PARAM_CONV, b, u.co, 3, 3, u.co, &u.w2);
      add_param(m, FDG_PARAM_BN_GAMMA, b, u.co, 1, 1, 1, &u.g2); add_param(m, FDG_PARAM_BN_BETA, b, u.co, 1, 1, 1, &u.b2);
      if (u.proj) {
        add_param(m, FDG_PARAM_CONV, b, u.co, 1, 1, u.ci, &u.ws);
        add_param(m, FDG_PARAM_BN_GAMMA, b, u.co, 1, 1, 1, &u.gs); add_param(m, FDG_PARAM_BN_BETA, b, u.co, 1, 1, 1, &u.bs);
      }
      u.r1 = add_running(m, u.co); u.r2 = add_running(m, u.co);
      if (u.proj) u.rs = add_running(m, u.co);
    } else {
      add_param(m, FDG_PARAM_BN_GAMMA, b, u.ci, 1, 1, 1, &u.g1); add_param(m, FDG_PARAM_BN_BETA, b, u.ci, 1, 1, 1, &u.b1);
      add_param(m, FDG_PARAM_CONV, b, u.co, 3, 3, u.ci, &u.w1);
      add_param(m, FDG_PARAM_BN_GAMMA, b, u.co, 1, 1, 1, &u.g2); add_param(m, FDG_PARAM_BN_BETA, b, u.co, 1, 1, 1, &u.b2);
      add_param(m, FDG_PARAM_CONV, b, u.co, 3, 3, u.co, &u.w2);
      if (u.proj) add_param(m, FDG_PARAM_CONV, b, u.co, 1, 1, u.ci, &u.ws);
      u.r1 = add_running(m, u.ci); u.r2 = add_running(m, u.co);
    }
    m.units.push_back(u);
    H = u.P; W = u.Q; ci = u.co;
  }
  {   // head
    Module& m = c->mods[K - 1];
    Unit u{}; u.type = U_HEAD; u.index = -1; u.ci = ci; u.co = a.num_classes; u.bn = wrn; u.H = H; u.W = W; u.P = 1; u.Q = 1; u.stride = 1;
    if (u.bn) { add_param(m, FDG_PARAM_BN_GAMMA, -1, ci, 1, 1, 1, &u.g1); add_param(m, FDG_PARAM_BN_BETA, -1, ci, 1, 1, 1, &u.b1); u.r1 = add_running(m, ci); }
    add_param(m, FDG_PARAM_FC_W, -1, a.num_classes, ci, 1, 1, &u.w1);
    add_param(m, FDG_PARAM_FC_B, -1, a.num_classes, 1, 1, 1, &u.w2);
    m.units.push_back(u);
  }
  // per-module slot layouts, depths and scratch sizes
  const size_t B = a.batch;
  for (int kk = 0; kk < K; ++kk) {
    Module& m = c->mods[kk];
    const int kp = kk + 1;
    m.D = (kp == K) ? 1 : 2 * (K - kp) + (c->cfg.order == FDG_FORWARD_FIRST ? 1 : 0);
    m.Dw = (kp == K) ? 1 : 2 * (K - kp) + 1;
    m.Din = (kp == 1) ? m.D + 2 : 0;
    if (c->use_graphs) {      // powers of two, so that every ring's phase is a function of t mod period
      m.D = pow2_at_least(m.D); m.Dw = pow2_at_least(m.Dw);
      if (m.Din) m.Din = pow2_at_least(m.Din);
      c->period = std::max(c->period, std::max(m.D, std::max(m.Dw, m.Din)));
    }
    m.in_elems = B * m.in_h * m.in_w * m.in_c;
    size_t te = 0, tf = 0, maxa = m.in_elems, scr = 0, wscr = 0;
    auto tens = [&](size_t e) { size_t o = te; te += align_up(e, 128); maxa = std::max(maxa, e); return o; };
    auto stat = [&](int ch) { size_t o = tf; tf += align_up((size_t)2 * ch, 64); return o; };
    auto red_scratch = [&](size_t rows, int ch) { scr = std::max(scr, (size_t)kRedMaxBlocks * kRedMaxSums * ch); (void)rows; };
    auto wg_scratch = [&](int n, int h, int w, int cin, int p, int q, int cout, int r, int stride, int pad) {
      ConvGeom g{n, h, w, cin, p, q, cout, r, r, stride, pad};
      wscr = std::max(wscr, conv_wgrad_scratch_elems(c->bf16_mode, g));
    };
    for (Unit& u : m.units) {
      const size_t in_e = B * u.H * u.W * u.ci, out_e = B * u.P * u.Q * u.co;
      maxa = std::max(maxa, std::max(in_e, out_e));
      switch (u.type) {
        case U_STEM:
          if (u.bn) { u.t_a = tens(out_e); u.st1 = stat(u.co); red_scratch(B * u.P * u.Q, u.co); }
          u.t_y = tens(out_e);
          wg_scratch(a.batch, u.H, u.W, u.ci, u.P, u.Q, u.co, 3, 1, 1);
          break;
        case U_BASIC:
          u.t_a = tens(out_e); u.t_b = tens(out_e); u.t_c = tens(out_e); u.t_y = tens(out_e);
          u.st1 = stat(u.co); u.st2 = stat(u.co);
          if (u.proj) { u.t_s = tens(out_e); u.sts = stat(u.co); }
          red_scratch(B * u.P * u.Q, u.co);
          wg_scratch(a.batch, u.H, u.W, u.ci, u.P, u.Q, u.co, 3, u.stride, 1);
          wg_scratch(a.batch, u.P, u.Q, u.co, u.P, u.Q, u.co, 3, 1, 1);
          if (u.proj) wg_scratch(a.batch, u.H, u.W, u.ci, u.P, u.Q, u.co, 1, u.stride, 0);
          break;
        case U_PREACT:
          u.t_a = tens(in_e); u.t_b = tens(out_e); u.t_c = tens(out_e); u.t_y = tens(out_e);
          u.st1 = stat(u.ci); u.st2 = stat(u.co);
          red_scratch(B * u.H * u.W, std::max(u.ci, u.co));
          wg_scratch(a.batch, u.H, u.W, u.ci, u.P, u.Q, u.co, 3, u.stride, 1);
          wg_scratch(a.batch, u.P, u.Q, u.co, u.P, u.Q, u.co, 3, 1, 1);
          if (u.proj) wg_scratch(a.batch, u.H, u.W, u.ci, u.P, u.Q, u.co, 1, u.stride, 0);
          break;
        case U_HEAD:
          if (u.bn) { u.t_a = tens(in_e); u.st1 = stat(u.ci); red_scratch(B * u.H * u.W, u.ci); }
          break;
      }
    }
    if (c->bf16_mode)
      for (const Unit& u : m.units) {
        if ((u.type != U_BASIC && u.type != U_PREACT) || u.stride != 2) continue;
        ConvGeom g1{a.batch, u.H, u.W, u.ci, u.P, u.Q, u.co, 3, 3, u.stride, 1};
        if (s2_uses_spread_dy(g1))
          m.up_elems = std::max(m.up_elems, B * u.H * u.W * u.co);
      }
    if (c->bf16_mode) {
      size_t fe = 0;
      auto flip = [&](size_t src, int co, int ci, int taps = 9) {
        tc::FlipEntry e; e.src = src; e.dst = fe; e.Co = co; e.Ci = ci; e.taps = taps;
        m.flip_table.push_back(e);
        long long off = (long long)fe;
        fe += align_up((size_t)co * taps * ci, 64);
        return off;
      };
      for (Unit& u : m.units) {
        if (u.type != U_BASIC && u.type != U_PREACT) continue;
        ConvGeom g1{a.batch, u.H, u.W, u.ci, u.P, u.Q, u.co, 3, 3, u.stride, 1};
        ConvGeom g2{a.batch, u.P, u.Q, u.co, u.P, u.Q, u.co, 3, 3, 1, 1};
        if (dgrad_uses_flipped(g1)) u.f1 = flip(u.w1, u.co, u.ci);
        if (dgrad_uses_flipped(g2)) u.f2 = flip(u.w2, u.co, u.co);
        if (u.proj) {
          ConvGeom gs{a.batch, u.H, u.W, u.ci, u.P, u.Q, u.co, 1, 1, u.stride, 0};
          if (dgrad_uses_flipped(gs)) u.fs = flip(u.ws, u.co, u.ci, 1);
        }
      }
      m.flip_elems = fe;
      size_t largest = 0;
      for (const tc::FlipEntry& fe_ : m.flip_table) largest = std::max(largest, (size_t)fe_.Co * fe_.taps * fe_.Ci);
      m.flip_blocks = (unsigned)std::min<size_t>(std::max<size_t>(largest / 8192, 8), 128);
    }
    m.slot_elems = te; m.slot_floats = tf; m.max_act = maxa; m.scratch_floats = scr; m.wscratch_floats = wscr;
    for (const Unit& u : m.units) {     // where the inference pass finds each batch norm's statistics
      const int c1 = (u.type == U_PREACT || u.type == U_HEAD) ? u.ci : u.co;
      if (u.r1 >= 0) m.eval_table.push_back(EvalStatEntry{(size_t)u.r1, u.st1, c1});
      if (u.r2 >= 0) m.eval_table.push_back(EvalStatEntry{(size_t)u.r2, u.st2, u.co});
      if (u.rs >= 0) m.eval_table.push_back(EvalStatEntry{(size_t)u.rs, u.sts, u.co});
    }
    {   // the gradient tensors a capture keeps (fdg_capture_begin), one region each
      size_t ce = 0;
      auto cap = [&](int ui, int which, size_t e, int ch) { m.cap_table.push_back(CaptureEntry{ui, which, ch, ce, e}); ce += align_up(e, 128); };
      for (int ui = 0; ui < (int)m.units.size(); ++ui) {
        const Unit& u = m.units[ui];
        const size_t in_e = B * u.H * u.W * u.ci, out_e = B * u.P * u.Q * u.co;
        if (u.type == U_STEM) { cap(ui, 0, out_e, u.co); if (u.bn) cap(ui, 3, out_e, u.co); }
        if (u.type == U_BASIC) {
          cap(ui, 0, out_e, u.co); cap(ui, 1, out_e, u.co); cap(ui, 2, out_e, u.co); cap(ui, 3, out_e, u.co); cap(ui, 4, in_e, u.ci);
          if (u.proj) cap(ui, 5, out_e, u.co);
        }
        if (u.type == U_PREACT) {
          cap(ui, 0, out_e, u.co); cap(ui, 1, out_e, u.co); cap(ui, 2, out_e, u.co); cap(ui, 3, in_e, u.ci); cap(ui, 4, in_e, u.ci);
          if (u.proj) cap(ui, 5, in_e, u.ci);
        }
      }
      m.cap_elems = ce;
    }
    const Unit& last = m.units.back();
    if (kp < K) { m.out_elems = B * last.P * last.Q * last.co; m.out_c = last.co; }
    m.slot_version.assign(m.D, -1);
    m.slot_batch.assign(m.D, -1);
  }
}

// Assigns every device pointer; with base == nullptr only measures.
static size_t carve(fdg_ctx* c, char* base) {
  Carver cv(base);
  c->guard_offsets.clear();
  cv.guards = &c->guard_offsets;
  const size_t es = c->esize;
  c->flags = cv.take<int>(256);
  c->tc_error = c->flags ? c->flags + 2 : nullptr;
  c->label_ring = c->use_graphs ? pow2_at_least(c->K + 2) : 2 * c->K + 2;
  c->mail_ring = c->use_graphs ? 4 : 3;
  if (c->use_graphs) c->period = std::max(c->period, std::max(c->label_ring, c->mail_ring));
  c->lr_dev = cv.take<float>(256);
  c->labels = cv.take<int32_t>((size_t)c->label_ring * c->arch.batch * sizeof(int32_t));
  size_t stage = 0;
  for (Module& m : c->mods) {
    m.theta = cv.take<float>(m.n_params * 4);
    m.mom = cv.take<float>(m.n_params * 4);
    m.grad = cv.take<float>(m.n_params * 4);
    m.wver = cv.take<float>((size_t)m.Dw * align_up(m.n_params, 64) * 4);
    m.wver16 = c->bf16_mode ? cv.take<bf16>((size_t)m.Dw * align_up(m.n_params, 64) * 2) : nullptr;
    m.wflip16 = m.flip_elems ? cv.take<bf16>((size_t)m.Dw * m.flip_elems * 2) : nullptr;
    m.flip_table_dev = m.flip_table.empty() ? nullptr : cv.take<tc::FlipEntry>(m.flip_table.size() * sizeof(tc::FlipEntry));
    // one slot beyond the FIFO's (and the image ring's) own: the inference pass works there
    m.fifo = cv.take<char>((size_t)(m.D + 1) * m.slot_elems * es);
    m.fifo_f = cv.take<float>((size_t)(m.D + 1) * std::max<size_t>(m.slot_floats, 64) * 4);
    m.in_ring = m.Din ? cv.take<char>((size_t)(m.Din + 1) * align_up(m.in_elems, 128) * es) : nullptr;
    m.running = cv.take<float>(std::max<size_t>(m.n_running, 64) * 4);
    m.eval_table_dev = m.eval_table.empty() ? nullptr : cv.take<EvalStatEntry>(m.eval_table.size() * sizeof(EvalStatEntry));
    m.mail = m.k >= 2 ? cv.take<char>((size_t)c->mail_ring * align_up(m.in_elems, 128) * es) : nullptr;
    for (int i = 0; i < 6; ++i) m.temps[i] = cv.take<char>(align_up(m.max_act, 128) * es);
    m.scratch = cv.take<float>(std::max<size_t>(m.scratch_floats, 64) * 4);
    m.wscratch = cv.take<float>(std::max<size_t>(m.wscratch_floats, 64) * 4);
    int maxc = 1;
    for (const Unit& u : m.units) maxc = std::max(maxc, std::max(u.ci, u.co));
    m.bnsums = cv.take<float>((size_t)kRedMaxSums * maxc * 4);
    m.counter = cv.take<unsigned int>(256);
    m.up = m.up_elems ? cv.take<char>(align_up(m.up_elems, 128) * es) : nullptr;
    {
      int widest = 64;                        // rows of 2 * C floats: narrow layers up to 64 channels, wide ones up to 640
      for (const Unit& u : m.units) if (u.type != U_HEAD && u.co <= tc::kStatChunks * 16) widest = std::max(widest, u.co);
      m.red_partial_floats = (size_t)kRedPartialCtas * 2 * widest;
      m.red_partial = cv.take<float>(m.red_partial_floats * 4);
    }
    m.red_counter = cv.take<unsigned int>(256);
    if (m.k == c->K) {
      const Unit& h = m.units.back();
      m.pooled = cv.take<float>((size_t)c->arch.batch * h.ci * 4);
      m.dlogits = cv.take<float>((size_t)c->arch.batch * h.co * 4);
      m.loss_n = cv.take<float>((size_t)c->arch.batch * 4);
      m.loss = cv.take<float>(256);
    }
    stage = std::max(stage, m.max_act);
  }
  c->host_images = cv.take<float>((size_t)c->arch.batch * c->arch.in_h * c->arch.in_w * c->arch.in_c * 4);
  c->host_labels = cv.take<int32_t>((size_t)c->arch.batch * 4);
  c->staging_elems = stage;
  c->staging = cv.take<float>(stage * 4);
  c->guard_table = cv.take<unsigned long long>((cv.count + 1) * sizeof(unsigned long long));   // one entry per buffer, itself included
  return align_up(cv.off, 256);
}

// ------------------------------------------------------------------ launching --
struct Launch {
  fdg_ctx* c;
  cudaStream_t st;
  cudaError_t err = cudaSuccess;
  int open_pair = -1;
  // begin/check bracket one kernel (or one kernel plus its fixed-order reduction): `bytes` and
  // `flops` are the algorithmic traffic and arithmetic of the launch, for roofline reports.
  void begin(int cls, double bytes, double flops) {
    open_pair = -1;
    if (!c->profiling || c->prof_recs.size() >= kProfMaxPairs) return;
    const size_t i = c->prof_recs.size();
    while (c->prof_events.size() < 2 * (i + 1)) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return;
      c->prof_events.push_back(e);
    }
    c->prof_recs.push_back(ProfRec{cls, bytes, flops});
    open_pair = (int)i;
    cudaEventRecord(c->prof_events[2 * i], st);
  }
  void end_events() {
    if (open_pair >= 0) cudaEventRecord(c->prof_events[2 * open_pair + 1], st);
    open_pair = -1;
  }
  void check() { if (err == cudaSuccess) err = cudaGetLastError(); ++c->launches; end_events(); }
  void note(cudaError_t e) { if (err == cudaSuccess) err = e; end_events(); }
};

// `run`: offset of this batch norm's running statistics in the module's vector (the kernel that forms the
// batch statistics also folds them into the running ones).
template <typename T>
static void bn_stats(Launch& L, Module& m, const T* x, size_t rows, int C, float eps, float* stats, long long run) {
  L.begin(KC_BN_STATS, (double)rows * C * sizeof(T), 3.0 * rows * C);
  L.note(launch_bn_stats<T>(L.st, x, rows, C, eps, stats, m.scratch, m.counter, run >= 0 ? m.running + run : nullptr, kBnMomentum));
  ++L.c->launches;
}

// `nparts` > 0: the statistics are not in `stats` yet; the convolution that produced x left nparts
// rows of partial sums in m.red_partial, which the kernel adds up first (and saves to `stats`).
template <typename T>
static void bn_apply(Launch& L, Module& m, const T* x, float* stats, const float* gamma, const float* beta, const T* res,
                     const float* res_stats, const float* res_gamma, const float* res_beta, bool relu, T* y,
                     size_t rows, int C, int nparts = 0, long long run = -1) {
  if (nparts < 0) nparts = 0;               // the statistics were finalised behind the convolution
  const size_t n = rows * C;
  L.begin(KC_BN_APPLY, (double)n * sizeof(T) * (res ? 3 : 2), 6.0 * n);
  L.note(launch_bn_apply<T>(L.st, x, stats, gamma, beta, res, res_stats, res_gamma, res_beta, relu, y, rows, C,
                            L.c->arch.bn_eps, nparts > 0 ? m.red_partial : nullptr, nparts, L.c->ew_block_cap,
                            (nparts > 0 && run >= 0) ? m.running + run : nullptr, kBnMomentum));
  ++L.c->launches;
}

// Backward of y = BN(x) (and optionally y2 = BN2(x2) sharing the same upstream gradient):
// dz = dy*[mask>0]; parameter gradients into dgamma/dbeta; dx (+res) and dx2.
template <typename T>
static void bn_backward(Launch& L, Module& m, const T* dy, const T* mask, const T* x, const float* stats,
                        const float* gamma, float* dgamma, float* dbeta, const T* x2, const float* stats2,
                        const float* gamma2, float* dgamma2, float* dbeta2, const T* res, T* dx, T* dx2,
                        size_t rows, int C, int nparts = 0) {
  const bool two = x2 != nullptr;
  const bool sums_ready = nparts > 0;    // the kernel that produced dy left nparts rows of partial sums in m.red_partial
  if (!sums_ready) {
    L.begin(KC_BN_BWD_REDUCE, (double)rows * C * sizeof(T) * (2 + (mask ? 1 : 0) + (two ? 1 : 0)), 8.0 * rows * C);
    L.note(launch_bn_bwd_reduce<T>(L.st, dy, mask, x, stats, x2, stats2, rows, C, m.bnsums, dgamma, dbeta, dgamma2, dbeta2,
                                   m.scratch, m.counter));
    ++L.c->launches;
  }
  const size_t n = rows * C;
  L.begin(KC_BN_BWD_APPLY, (double)n * sizeof(T) * (3 + (mask ? 1 : 0) + (two ? 2 : 0) + (res ? 1 : 0)), 10.0 * n);
  L.note(launch_bn_bwd_apply<T>(L.st, dy, mask, x, stats, gamma, m.bnsums, x2, stats2, gamma2, res, dx, dx2, rows, C,
                                sums_ready ? m.red_partial : nullptr, nparts, dgamma, dbeta, L.c->ew_block_cap));
  ++L.c->launches;
}

template <typename T>
static void scale_tensor(Launch& L, const T* in, T* out, float s, size_t n) {
  L.begin(KC_SHRINK, 2.0 * n * sizeof(T), (double)n);
  L.note(launch_scale<T>(L.st, in, out, s, n));
  ++L.c->launches;
}

template <typename T> static const T* weights_of(const Module& m, int vslot);
template <> const float* weights_of<float>(const Module& m, int vslot) { return m.wver + (size_t)vslot * align_up(m.n_params, 64); }
template <> const bf16* weights_of<bf16>(const Module& m, int vslot) { return m.wver16 + (size_t)vslot * align_up(m.n_params, 64); }

static ConvGeom geom(int N, int H, int W, int Ci, int P, int Q, int Co, int R, int stride, int pad) {
  return ConvGeom{N, H, W, Ci, P, Q, Co, R, R, stride, pad};
}

static double conv_flops(const ConvGeom& g) { return 2.0 * g.N * g.P * g.Q * g.Co * (double)g.R * g.S * g.Ci; }
static double in_elems(const ConvGeom& g) { return (double)g.N * g.H * g.W * g.Ci; }
static double out_elems(const ConvGeom& g) { return (double)g.N * g.P * g.Q * g.Co; }
static double w_elems(const ConvGeom& g) { return (double)g.Co * g.R * g.S * g.Ci; }

// `want_stats`: the caller will batch-normalise y.  Returns the number of rows of per-channel partial
// sums (sum y, sum y^2) the convolution kernel left in m.red_partial from its epilogue, or 0 when it
// left none and the caller has to run bn_stats.
template <typename T>
// Returns the rows of partial sums the kernel left in m.red_partial for the batch norm that follows (`want_stats`;
// a narrow layer), 0 when it formed none, or -1 when the statistics are already in `stats` (a wide layer, whose
// totals are finalised right behind the convolution; needs `stats`, with `run` the running statistics' offset or -1).
static int conv_fprop(Launch& L, Module& m, const ConvGeom& g, const T* x, const T* w, T* y, const T* res,
                      bool want_stats = false, float* stats = nullptr, long long run = -1) {
  L.begin(KC_CONV_FPROP, (in_elems(g) + w_elems(g) + out_elems(g) * (res ? 2 : 1)) * sizeof(T), conv_flops(g));
  int nparts = 0;
  if constexpr (std::is_same<T, bf16>::value) {
    halo::EpiReduce r{};
    r.mode = 1; r.partial = m.red_partial;
    const WideStats ws{m.red_partial, m.red_partial_floats, stats, (size_t)g.N * g.P * g.Q, L.c->arch.bn_eps,
                       run >= 0 ? m.running + run : nullptr, kBnMomentum};
    L.note(bf16_conv_fprop(L.st, &L.c->tmaps, g, x, w, y, res, want_stats ? &r : nullptr, &nparts, L.c->tc_error, &L.c->launches,
                           (want_stats && stats) ? &ws : nullptr));
  } else {
    L.note(launch_conv_simt<T, CONV_FPROP>(L.st, g, x, w, y, nullptr, nullptr, res, (const T*)nullptr, &L.c->launches));
  }
  return nparts;
}
// `wflip` is the flipped/transposed weight copy (bf16 mode, tensor-core eligible shapes) or null.
// The batch-norm backward that will consume dx as its upstream gradient: dz = dx * [mask > 0],
// xhat from (x, stats).  When the data-gradient kernel can, it forms that backward's two sums
// per CTA in its epilogue and conv_dgrad returns the number of partial rows left in m.red_partial.
template <typename T> struct NextBnBwd { const T* mask; const T* x; const float* stats; };

template <typename T>
static int conv_dgrad(Launch& L, Module& m, const ConvGeom& g, const T* dy, const T* w, const T* wflip, T* dx,
                       const T* res, const T* mask, const NextBnBwd<T>* next = nullptr, const T* dy_up = nullptr) {
  L.begin(KC_CONV_DGRAD, (out_elems(g) + w_elems(g) + in_elems(g) * (1 + (res ? 1 : 0) + (mask ? 1 : 0) + (next ? 2 : 0))) * sizeof(T), conv_flops(g));
  int nparts = 0;
  if constexpr (std::is_same<T, bf16>::value) {
    halo::EpiReduce r{};
    if (next) { r.mode = 2; r.mask = next->mask; r.xprev = next->x; r.pstats = next->stats; r.partial = m.red_partial; }
    L.note(bf16_conv_dgrad(L.st, &L.c->tmaps, g, dy, w, wflip, dy_up, dx, res, mask, next ? &r : nullptr, &nparts, L.c->tc_error, &L.c->launches));
  } else {
    L.note(launch_conv_simt<T, CONV_DGRAD>(L.st, g, dy, w, dx, nullptr, nullptr, res, mask, &L.c->launches));
  }
  return nparts;
}
template <typename T>
static void conv_wgrad(Launch& L, Module& m, const ConvGeom& g, const T* x, const T* dy, float* dw, const T* dy_up = nullptr) {
  L.begin(KC_CONV_WGRAD, (in_elems(g) + out_elems(g)) * sizeof(T) + w_elems(g) * 4, conv_flops(g));
  // the tensor-core and small-shape kernels serve bf16 storage only: the fp32 mode keeps one summation
  // scheme for all its weight gradients
  if constexpr (std::is_same<T, bf16>::value)
    L.note(bf16_conv_wgrad(L.st, &L.c->tmaps, g, x, dy, dy_up, dw, m.wscratch, L.c->tc_error, L.st == m.stream2, &L.c->launches));
  else
    L.note(launch_conv_simt<T, CONV_WGRAD>(L.st, g, x, dy, (T*)nullptr, m.wscratch, dw, (const T*)nullptr, (const T*)nullptr, &L.c->launches));
}

template <typename T> static const T* flipped_of(const Module& m, int vslot, long long off);
template <> const float* flipped_of<float>(const Module&, int, long long) { return nullptr; }
template <> const bf16* flipped_of<bf16>(const Module& m, int vslot, long long off) {
  return off < 0 ? nullptr : m.wflip16 + (size_t)vslot * m.flip_elems + off;
}

// dy [N][P][Q][Co] of a stride-2 convolution, spread onto the even pixels of a zero [N][H][W][Co] tensor
// (module scratch); null when the stride-2 gradients of this shape stay on the CUDA cores.
template <typename T>
static const T* upsample_dy(Launch& L, Module& m, const ConvGeom& g, const T* dy) {
  if constexpr (std::is_same<T, bf16>::value) {
    if (!m.up || !s2_uses_spread_dy(g)) return nullptr;
    T* up = reinterpret_cast<T*>(m.up);
    L.begin(KC_CONV_DGRAD, (double)g.N * g.H * g.W * g.Co * 2 * 1.25, 0.0);
    L.note(bf16_spread_dy(L.st, g, dy, up, &L.c->launches));
    return up;
  }
  return nullptr;
}

// ------------------------------------------------------------ module passes ---
template <typename T> static T* slot_T(const Module& m, int slot) { return reinterpret_cast<T*>(m.fifo) + (size_t)slot * m.slot_elems; }
static float* slot_F(const Module& m, int slot) { return m.fifo_f + (size_t)slot * std::max<size_t>(m.slot_floats, 64); }

// Input tensor of module m for batch tau: the image ring (module 1) or the upstream module's FIFO slot.
// `eval`: the inference pass reads the extra slot behind each ring instead of batch tau's.
template <typename T>
static const T* module_input(fdg_ctx* c, const Module& m, int64_t tau, bool eval = false) {
  if (m.k == 1) return reinterpret_cast<const T*>(m.in_ring) + (size_t)(eval ? m.Din : tau % m.Din) * align_up(m.in_elems, 128);
  const Module& up = c->mods[m.k - 2];
  return slot_T<T>(up, eval ? up.D : (int)(tau % up.D)) + up.units.back().t_y;
}

// Forward of the module's units into FIFO slot `slot` with weight version `vslot`.  Training (`eval` false):
// batch statistics, formed in the convolution epilogues where the kernel can, saved for the backward and
// folded into the running statistics.  Inference (`eval` true): the statistics of every batch norm were put
// into the slot beforehand from the running ones (bn_eval_stats_kernel), nothing is reduced.
template <typename T>
static void forward_module(fdg_ctx* c, Module& m, Launch& L, int64_t tau, int slot, int vslot, bool eval = false) {
  const int B = c->arch.batch;
  const float eps = c->arch.bn_eps;
  const T* wt = weights_of<T>(m, vslot);
  const float* wf = m.wver + (size_t)vslot * align_up(m.n_params, 64);
  T* S = slot_T<T>(m, slot);
  float* F = slot_F(m, slot);
  const T* x = module_input<T>(c, m, tau, eval);
  T* tmp = reinterpret_cast<T*>(m.temps[2]);
  // statistics of a convolution output y that left `np` rows of partial sums (0: reduce y now)
  auto stats_of = [&](int np, const T* y, size_t rows, int C, float* stats, long long run) {
    if (!eval && np == 0) bn_stats<T>(L, m, y, rows, C, eps, stats, run);
  };
  int x_np = 0;     // -1: the statistics of x (the next pre-activation block's first batch norm) are already in place
  for (size_t ui = 0; ui < m.units.size(); ++ui) {
    const Unit& u = m.units[ui];
    // the pre-activation block that normalises this unit's output first, if it is in this module
    const Unit* nxt = (ui + 1 < m.units.size() && m.units[ui + 1].type == U_PREACT) ? &m.units[ui + 1] : nullptr;
    const size_t rows_in = (size_t)B * u.H * u.W, rows_out = (size_t)B * u.P * u.Q;
    switch (u.type) {
      case U_STEM: {
        ConvGeom g = geom(B, u.H, u.W, u.ci, u.P, u.Q, u.co, 3, 1, 1);
        if (u.bn) {
          const int np = conv_fprop<T>(L, m, g, x, wt + u.w1, S + u.t_a, nullptr, !eval, F + u.st1, u.r1);
          stats_of(np, S + u.t_a, rows_out, u.co, F + u.st1, u.r1);
          bn_apply<T>(L, m, S + u.t_a, F + u.st1, wf + u.g1, wf + u.b1, nullptr, nullptr, nullptr, nullptr, true, S + u.t_y, rows_out, u.co, np, u.r1);
        } else {
          conv_fprop<T>(L, m, g, x, wt + u.w1, S + u.t_y, nullptr);
        }
        break;
      }
      case U_BASIC: {
        ConvGeom g1 = geom(B, u.H, u.W, u.ci, u.P, u.Q, u.co, 3, u.stride, 1);
        ConvGeom g2 = geom(B, u.P, u.Q, u.co, u.P, u.Q, u.co, 3, 1, 1);
        const int np1 = conv_fprop<T>(L, m, g1, x, wt + u.w1, S + u.t_a, nullptr, !eval, F + u.st1, u.r1);   // c1
        stats_of(np1, S + u.t_a, rows_out, u.co, F + u.st1, u.r1);
        bn_apply<T>(L, m, S + u.t_a, F + u.st1, wf + u.g1, wf + u.b1, nullptr, nullptr, nullptr, nullptr, true, S + u.t_b, rows_out, u.co, np1, u.r1);  // a1
        if (u.proj) {          // shortcut first: its statistics must not disturb the partial sums conv2 leaves for BN2
          ConvGeom gs = geom(B, u.H, u.W, u.ci, u.P, u.Q, u.co, 1, u.stride, 0);
          const int nps = conv_fprop<T>(L, m, gs, x, wt + u.ws, S + u.t_s, nullptr, !eval, F + u.sts, u.rs);   // cs
          stats_of(nps < 0 ? nps : 0, S + u.t_s, rows_out, u.co, F + u.sts, u.rs);
        }
        const int np2 = conv_fprop<T>(L, m, g2, S + u.t_b, wt + u.w2, S + u.t_c, nullptr, !eval, F + u.st2, u.r2);   // c2
        stats_of(np2, S + u.t_c, rows_out, u.co, F + u.st2, u.r2);
        if (u.proj) {
          bn_apply<T>(L, m, S + u.t_c, F + u.st2, wf + u.g2, wf + u.b2, S + u.t_s, F + u.sts, wf + u.gs, wf + u.bs, true, S + u.t_y, rows_out, u.co, np2, u.r2);
        } else if (u.zpad) {   // the shortcut is x at every stride-th pixel between zero channels: built in a temporary
          L.begin(KC_BN_APPLY, (double)rows_out * (u.ci + u.co) * sizeof(T), 0.0);
          pad_shortcut_kernel<T><<<ew_blocks(rows_out * u.co), 256, 0, L.st>>>(x, tmp, rows_out, u.P, u.Q, u.H, u.W, u.ci, u.co, u.stride);
          L.check();
          bn_apply<T>(L, m, S + u.t_c, F + u.st2, wf + u.g2, wf + u.b2, tmp, nullptr, nullptr, nullptr, true, S + u.t_y, rows_out, u.co, np2, u.r2);
        } else {
          bn_apply<T>(L, m, S + u.t_c, F + u.st2, wf + u.g2, wf + u.b2, x, nullptr, nullptr, nullptr, true, S + u.t_y, rows_out, u.co, np2, u.r2);
        }
        break;
      }
      case U_PREACT: {
        ConvGeom g1 = geom(B, u.H, u.W, u.ci, u.P, u.Q, u.co, 3, u.stride, 1);
        ConvGeom g2 = geom(B, u.P, u.Q, u.co, u.P, u.Q, u.co, 3, 1, 1);
        stats_of(x_np, x, rows_in, u.ci, F + u.st1, u.r1);
        x_np = 0;
        bn_apply<T>(L, m, x, F + u.st1, wf + u.g1, wf + u.b1, nullptr, nullptr, nullptr, nullptr, true, S + u.t_a, rows_in, u.ci);   // o
        const int np = conv_fprop<T>(L, m, g1, S + u.t_a, wt + u.w1, S + u.t_b, nullptr, !eval, F + u.st2, u.r2);   // c1
        stats_of(np, S + u.t_b, rows_out, u.co, F + u.st2, u.r2);
        bn_apply<T>(L, m, S + u.t_b, F + u.st2, wf + u.g2, wf + u.b2, nullptr, nullptr, nullptr, nullptr, true, S + u.t_c, rows_out, u.co, np, u.r2); // a2
        if (u.proj) {
          ConvGeom gs = geom(B, u.H, u.W, u.ci, u.P, u.Q, u.co, 1, u.stride, 0);
          conv_fprop<T>(L, m, gs, S + u.t_a, wt + u.ws, tmp, nullptr);
          x_np = conv_fprop<T>(L, m, g2, S + u.t_c, wt + u.w2, S + u.t_y, tmp, !eval && nxt, nxt ? F + nxt->st1 : nullptr, nxt ? nxt->r1 : -1);
        } else {
          x_np = conv_fprop<T>(L, m, g2, S + u.t_c, wt + u.w2, S + u.t_y, x, !eval && nxt, nxt ? F + nxt->st1 : nullptr, nxt ? nxt->r1 : -1);
        }
        if (x_np > 0) x_np = 0;     // rows for a narrow layer's apply kernel: not used here, the block's input is reduced as before
        break;
      }
      case U_HEAD:
        break;      // handled by head_forward_backward / head_eval
    }
    if (u.type != U_HEAD) x = S + u.t_y;
  }
}

// Module K, inference: [BN + ReLU,] global average pool, FC, arg-max against the labels.
template <typename T>
static void head_eval(fdg_ctx* c, Module& m, Launch& L, int slot, int vslot, const int32_t* labels_dev, float* logits_dev,
                      int* correct_dev) {
  const Unit& u = m.units.back();
  const int B = c->arch.batch, F = u.ci, classes = u.co, HW = u.H * u.W;
  const float* wf = m.wver + (size_t)vslot * align_up(m.n_params, 64);
  T* S = slot_T<T>(m, slot);
  float* Fs = slot_F(m, slot);
  const T* x = m.units.size() >= 2 ? S + m.units[m.units.size() - 2].t_y : module_input<T>(c, m, 0, true);
  const T* feat = x;
  if (u.bn) {
    bn_apply<T>(L, m, x, Fs + u.st1, wf + u.g1, wf + u.b1, nullptr, nullptr, nullptr, nullptr, true, S + u.t_a, (size_t)B * HW, F);
    feat = S + u.t_a;
  }
  L.begin(KC_HEAD, (double)B * HW * F * sizeof(T), 2.0 * B * F * classes);
  head_eval_kernel<T><<<B, 128, (size_t)(F + classes) * 4, L.st>>>(feat, wf + u.w1, wf + u.w2, labels_dev, HW, F, classes,
                                                                  logits_dev, correct_dev);
  L.check();
}

// Module K only: classifier, loss and their backward; leaves the gradient of the last block's
// output in `gout`.
template <typename T>
static void head_forward_backward(fdg_ctx* c, Module& m, Launch& L, int64_t tau, int slot, int vslot, T* gout) {
  const Unit& u = m.units.back();
  const int B = c->arch.batch, F = u.ci, classes = u.co, HW = u.H * u.W;
  const float* wf = m.wver + (size_t)vslot * align_up(m.n_params, 64);
  T* S = slot_T<T>(m, slot);
  float* Fs = slot_F(m, slot);
  const T* x = m.units.size() >= 2 ? S + m.units[m.units.size() - 2].t_y : module_input<T>(c, m, tau);
  const size_t rows = (size_t)B * HW;
  const T* feat = x;
  if (u.bn) {
    bn_stats<T>(L, m, x, rows, F, c->arch.bn_eps, Fs + u.st1, u.r1);
    bn_apply<T>(L, m, x, Fs + u.st1, wf + u.g1, wf + u.b1, nullptr, nullptr, nullptr, nullptr, true, S + u.t_a, rows, F);
    feat = S + u.t_a;
  }
  const int32_t* labels = c->labels + (size_t)(tau % c->label_ring) * B;
  T* dfeat = u.bn ? reinterpret_cast<T*>(m.temps[2]) : gout;
  L.begin(KC_HEAD, 2.0 * rows * F * sizeof(T), 4.0 * B * F * classes);
  L.note(launch_head<T>(L.st, feat, wf + u.w1, wf + u.w2, labels, HW, F, classes, B, m.pooled, m.dlogits, m.loss_n, dfeat,
                        m.grad + u.w1, m.grad + u.w2, m.loss, c->flags, false, true));
  ++c->launches;
  L.begin(KC_HEAD, 4.0 * B * (F + classes) + 4.0 * classes * F, 2.0 * B * F * classes);
  L.note(launch_head<T>(L.st, feat, wf + u.w1, wf + u.w2, labels, HW, F, classes, B, m.pooled, m.dlogits, m.loss_n, dfeat,
                        m.grad + u.w1, m.grad + u.w2, m.loss, c->flags, true, false));
  ++c->launches;
  if (u.bn)
    bn_backward<T>(L, m, dfeat, feat, x, Fs + u.st1, wf + u.g1, m.grad + u.g1, m.grad + u.b1, nullptr, nullptr, nullptr,
                   nullptr, nullptr, nullptr, gout, nullptr, rows, F);
}

// Chain rule through the module's blocks (and stem) for the batch saved in `slot`.
//   gin   gradient with respect to the module output (already shrunk), consumed
//   gfirst where the gradient of the module input goes (mailbox slot; unused for module 1)
// `LS` issues on the module's side stream (the same stream as L when `forked` is false): the weight
// gradients run there, beside the chain batch-norm backward -> data gradient -> next layer.  Buffers
// a weight gradient reads (0: T1, 1: T4, 2: T2, 3: the spread-out dy) are not rewritten on the main
// stream before the event recorded behind their last reader.
template <typename T>
static void backward_module(fdg_ctx* c, Module& m, Launch& L, Launch& LS, bool forked, int64_t tau, int slot, int vslot,
                            T* gin, T* gfirst) {
  const int B = c->arch.batch;
  const T* wt = weights_of<T>(m, vslot);
  const float* wf = m.wver + (size_t)vslot * align_up(m.n_params, 64);
  T* S = slot_T<T>(m, slot);
  float* F = slot_F(m, slot);
  T* G[2] = {reinterpret_cast<T*>(m.temps[0]), reinterpret_cast<T*>(m.temps[1])};
  T* T1 = reinterpret_cast<T*>(m.temps[2]);
  T* T2 = reinterpret_cast<T*>(m.temps[3]);
  T* T3 = reinterpret_cast<T*>(m.temps[4]);
  T* T4 = reinterpret_cast<T*>(m.temps[5]);
  bool buf_read[4] = {false, false, false, false};
  bool side_used = false;
  auto fork = [&]() {
    if (!forked) return;
    side_used = true;
    L.note(cudaEventRecord(m.ev_fork2, L.st));
    LS.note(cudaStreamWaitEvent(LS.st, m.ev_fork2, 0));
  };
  auto side_done = [&](int b) { if (forked) { LS.note(cudaEventRecord(m.ev_buf[b], LS.st)); buf_read[b] = true; } };
  auto wait_buf = [&](int b) { if (forked && buf_read[b]) L.note(cudaStreamWaitEvent(L.st, m.ev_buf[b], 0)); };
  // While a capture is on (fdg_capture_begin), every gradient tensor of the pass is copied aside in stream order.
  auto keep = [&](int ui, int which, const T* src) {
    if (!m.cap_buf || !src) return;
    for (const CaptureEntry& ce : m.cap_table)
      if (ce.unit == ui && ce.which == which) {
        L.note(cudaMemcpyAsync(m.cap_buf + ce.off * sizeof(T), src, ce.elems * sizeof(T), cudaMemcpyDeviceToDevice, L.st));
        return;
      }
  };
  if (m.cap_buf) m.cap_batch = tau;
  T* dy = gin;
  int dy_sum_parts = 0;            // > 0: the kernel that produced dy left that many rows of partial sums for the
                                   // first batch-norm backward it meets
  const int nu = (int)m.units.size();
  for (int i = nu - 1; i >= 0; --i) {
    const Unit& u = m.units[i];
    if (u.type == U_HEAD) continue;
    const T* x = i > 0 ? S + m.units[i - 1].t_y : module_input<T>(c, m, tau);
    T* gout = (i == 0) ? gfirst : (dy == G[0] ? G[1] : G[0]);
    const size_t rows_in = (size_t)B * u.H * u.W, rows_out = (size_t)B * u.P * u.Q;
    // The batch-norm backward that unit i-1 will start with, if its sums can be formed by the
    // data-gradient kernel that writes this unit's input gradient.
    NextBnBwd<T> nb{};
    const NextBnBwd<T>* next = nullptr;
    if (i > 0) {
      const Unit& pu = m.units[i - 1];
      if (pu.type == U_BASIC && !pu.proj) { nb = {S + pu.t_y, S + pu.t_c, F + pu.st2}; next = &nb; }
      if (pu.type == U_STEM && pu.bn) { nb = {S + pu.t_y, S + pu.t_a, F + pu.st1}; next = &nb; }
    }
    int out_sum_parts = 0;
    switch (u.type) {
      case U_STEM: {
        ConvGeom g = geom(B, u.H, u.W, u.ci, u.P, u.Q, u.co, 3, 1, 1);
        const T* dc = dy;
        keep(i, 0, dy);
        if (u.bn) {
          wait_buf(0);
          bn_backward<T>(L, m, dy, S + u.t_y, S + u.t_a, F + u.st1, wf + u.g1, m.grad + u.g1, m.grad + u.b1, nullptr,
                         nullptr, nullptr, nullptr, nullptr, nullptr, T1, nullptr, rows_out, u.co, dy_sum_parts);
          dc = T1;
          keep(i, 3, T1);
        }
        fork();
        conv_wgrad<T>(LS, m, g, x, dc, m.grad + u.w1);
        side_done(0);
        break;
      }
      case U_BASIC: {
        ConvGeom g1 = geom(B, u.H, u.W, u.ci, u.P, u.Q, u.co, 3, u.stride, 1);
        ConvGeom g2 = geom(B, u.P, u.Q, u.co, u.P, u.Q, u.co, 3, 1, 1);
        keep(i, 0, dy);
        wait_buf(0);
        if (u.proj) {
          wait_buf(2);
          bn_backward<T>(L, m, dy, S + u.t_y, S + u.t_c, F + u.st2, wf + u.g2, m.grad + u.g2, m.grad + u.b2, S + u.t_s,
                         F + u.sts, wf + u.gs, m.grad + u.gs, m.grad + u.bs, nullptr, T1, T2, rows_out, u.co);
        } else {
          bn_backward<T>(L, m, dy, S + u.t_y, S + u.t_c, F + u.st2, wf + u.g2, m.grad + u.g2, m.grad + u.b2, nullptr,
                         nullptr, nullptr, nullptr, nullptr, nullptr, T1, nullptr, rows_out, u.co, dy_sum_parts);
        }
        keep(i, 1, T1);
        if (u.proj) keep(i, 5, T2);
        fork();
        conv_wgrad<T>(LS, m, g2, S + u.t_b, T1, m.grad + u.w2);                                          // side
        side_done(0);
        const NextBnBwd<T> bn1{S + u.t_b, S + u.t_a, F + u.st1};
        const int bn1_parts = conv_dgrad<T>(L, m, g2, T1, wt + u.w2, flipped_of<T>(m, vslot, u.f2), T3, nullptr, nullptr, &bn1);   // da1
        keep(i, 2, T3);
        wait_buf(1);
        bn_backward<T>(L, m, T3, S + u.t_b, S + u.t_a, F + u.st1, wf + u.g1, m.grad + u.g1, m.grad + u.b1, nullptr,
                       nullptr, nullptr, nullptr, nullptr, nullptr, T4, nullptr, rows_out, u.co, bn1_parts);      // dc1
        keep(i, 3, T4);
        const T* up = nullptr;
        if (u.stride == 2) { wait_buf(3); up = upsample_dy<T>(L, m, g1, T4); }
        fork();
        conv_wgrad<T>(LS, m, g1, x, T4, m.grad + u.w1, up);                                              // side
        side_done(1);
        if (up) side_done(3);
        const bool need_dx = !(m.k == 1 && i == 0);
        if (u.proj) {
          ConvGeom gs = geom(B, u.H, u.W, u.ci, u.P, u.Q, u.co, 1, u.stride, 0);
          conv_wgrad<T>(LS, m, gs, x, T2, m.grad + u.ws);                                                // side
          side_done(2);
          if (need_dx) {
            conv_dgrad<T>(L, m, gs, T2, wt + u.ws, flipped_of<T>(m, vslot, u.fs), T3, nullptr, nullptr);
            out_sum_parts = conv_dgrad<T>(L, m, g1, T4, wt + u.w1, flipped_of<T>(m, vslot, u.f1), gout, T3, nullptr, next, up);
          }
        } else if (need_dx && u.zpad) {
          // the shortcut's share: the gated upstream gradient's middle channels, put back at every stride-th pixel
          L.begin(KC_BN_BWD_APPLY, (double)(rows_out * u.co * 2 + rows_in * u.ci) * sizeof(T), 0.0);
          pad_shortcut_bwd_kernel<T><<<ew_blocks(rows_in * u.ci), 256, 0, L.st>>>(dy, S + u.t_y, T3, rows_in, u.P, u.Q, u.H, u.W, u.ci, u.co, u.stride);
          L.check();
          out_sum_parts = conv_dgrad<T>(L, m, g1, T4, wt + u.w1, flipped_of<T>(m, vslot, u.f1), gout, T3, nullptr, next, up);
        } else if (need_dx) {
          out_sum_parts = conv_dgrad<T>(L, m, g1, T4, wt + u.w1, flipped_of<T>(m, vslot, u.f1), gout, dy, S + u.t_y, next);
        }
        if (need_dx) keep(i, 4, gout);
        break;
      }
      case U_PREACT: {
        ConvGeom g1 = geom(B, u.H, u.W, u.ci, u.P, u.Q, u.co, 3, u.stride, 1);
        ConvGeom g2 = geom(B, u.P, u.Q, u.co, u.P, u.Q, u.co, 3, 1, 1);
        keep(i, 0, dy);
        conv_wgrad<T>(L, m, g2, S + u.t_c, dy, m.grad + u.w2);
        conv_dgrad<T>(L, m, g2, dy, wt + u.w2, flipped_of<T>(m, vslot, u.f2), T1, nullptr, nullptr);   // da2
        keep(i, 1, T1);
        bn_backward<T>(L, m, T1, S + u.t_c, S + u.t_b, F + u.st2, wf + u.g2, m.grad + u.g2, m.grad + u.b2, nullptr,
                       nullptr, nullptr, nullptr, nullptr, nullptr, T2, nullptr, rows_out, u.co);      // dc1
        keep(i, 2, T2);
        const T* up = u.stride == 2 ? upsample_dy<T>(L, m, g1, T2) : nullptr;
        conv_wgrad<T>(L, m, g1, S + u.t_a, T2, m.grad + u.w1, up);
        if (u.proj) {
          ConvGeom gs = geom(B, u.H, u.W, u.ci, u.P, u.Q, u.co, 1, u.stride, 0);
          conv_wgrad<T>(L, m, gs, S + u.t_a, dy, m.grad + u.ws);
          conv_dgrad<T>(L, m, gs, dy, wt + u.ws, flipped_of<T>(m, vslot, u.fs), T3, nullptr, nullptr);
          keep(i, 5, T3);
          conv_dgrad<T>(L, m, g1, T2, wt + u.w1, flipped_of<T>(m, vslot, u.f1), T1, T3, nullptr, nullptr, up);   // do
        } else {
          conv_dgrad<T>(L, m, g1, T2, wt + u.w1, flipped_of<T>(m, vslot, u.f1), T1, nullptr, nullptr);
        }
        keep(i, 3, T1);
        bn_backward<T>(L, m, T1, S + u.t_a, x, F + u.st1, wf + u.g1, m.grad + u.g1, m.grad + u.b1, nullptr, nullptr,
                       nullptr, nullptr, nullptr, u.proj ? nullptr : dy, gout, nullptr, rows_in, u.ci);
        keep(i, 4, gout);
        break;
      }
      default: break;
    }
    dy = gout;
    dy_sum_parts = out_sum_parts;
  }
  if (forked && side_used) {      // every parameter gradient is in place before the update that follows
    LS.note(cudaEventRecord(m.ev_join2, LS.st));
    L.note(cudaStreamWaitEvent(L.st, m.ev_join2, 0));
  }
}

template <typename T>
static void update_module(fdg_ctx* c, Module& m, Launch& L, int next_vslot) {
  const size_t n = m.n_params;
  float* next32 = m.wver + (size_t)next_vslot * align_up(n, 64);
  bf16* next16 = c->bf16_mode ? m.wver16 + (size_t)next_vslot * align_up(n, 64) : nullptr;
  L.begin(KC_SGD, (double)n * (24 + (next16 ? 2 : 0)), 6.0 * n);
  L.note(launch_sgd(L.st, m.theta, m.mom, m.grad, next32, next16, n, c->lr, c->graph_mode_entered ? c->lr_dev : nullptr,
                    c->cfg.momentum, c->cfg.weight_decay));
  ++c->launches;
  if (m.flip_table_dev) {
    L.begin(KC_SGD, 4.0 * m.flip_elems, 0.0);
    tc::wflip_kernel<<<dim3(m.flip_blocks, (unsigned)m.flip_table.size()), 256, 0, L.st>>>(next16, m.wflip16 + (size_t)next_vslot * m.flip_elems, m.flip_table_dev);
    L.check();
  }
}

// How a module-step is issued.
//   STREAMS  on the module's own stream, ordered against its neighbours by the events of iteration t-1
//   SERIAL   on the caller's stream, modules one after the other
//   CAPTURE  on the module's own stream while an iteration is being recorded into a graph: the
//            iteration's graph follows the previous iteration's on the caller's stream, so nothing has
//            to be waited for; the loss is copied by the caller afterwards
//   DRY      nothing is enqueued; only the host-side bookkeeping advances (a recorded graph is replayed)
enum StepMode { RUN_STREAMS, RUN_SERIAL, RUN_CAPTURE, RUN_DRY };

// One module-step of module m in iteration t (Algorithm I, body of "Parallel for k").
template <typename T>
static cudaError_t module_step(fdg_ctx* c, Module& m, cudaStream_t st, StepMode mode, float* loss_dev) {
  const int K = c->K, k = m.k;
  const int64_t t = c->t;
  const int64_t tau_f = t - k + 1, tau_b = t - 2 * (int64_t)K + k + 1;
  const int e_prev = (int)((t - 1) % kEventRing), e_now = (int)(t % kEventRing);
  const bool events = mode == RUN_STREAMS, enqueue = mode != RUN_DRY;
  Launch L{c, st};
  fdg_sched_entry row;
  row.t = t; row.k = k; row.tau_f = row.tau_b = row.ver_f = row.ver_b = -1; row.slot_f = row.slot_b = -1;
  auto sig = [&](int64_t v) { c->step_sig = c->step_sig * 1000003ull + (uint64_t)(v + 7); };

  auto wait_act = [&]() {
    if (!events) return;
    if (k == 1) L.note(cudaStreamWaitEvent(st, c->ev_in[e_now], 0));
    else L.note(cudaStreamWaitEvent(st, c->mods[k - 2].ev_act[e_prev], 0));
  };
  auto wait_grad = [&]() {
    if (!events || k == K) return;
    L.note(cudaStreamWaitEvent(st, c->mods[k].ev_grad[e_prev], 0));
  };
  auto do_forward = [&]() {
    if (tau_f < 1 || tau_f > c->last_batch) return;
    const int slot = (int)(tau_f % m.D), vslot = (int)(m.updates % m.Dw);
    if (enqueue) forward_module<T>(c, m, L, tau_f, slot, vslot);
    m.slot_version[slot] = m.updates; m.slot_batch[slot] = tau_f;
    row.tau_f = tau_f; row.ver_f = m.updates; row.slot_f = slot;
    sig(slot); sig(vslot); sig(k == 1 ? tau_f % m.Din : 0);
    if (k < K) { m.last_out_batch = tau_f; m.last_out_slot = slot; }
  };
  auto do_backward_update = [&]() {
    if (tau_b < 1 || tau_b > c->last_batch) return;
    const int slot = (int)(tau_b % m.D);
    const int64_t ver = (c->cfg.weight_reading == FDG_STASHED) ? m.slot_version[slot] : m.updates;
    const int vslot = (int)(ver % m.Dw);
    const int next_vslot = (int)((m.updates + 1) % m.Dw);
    sig(slot); sig(vslot); sig(next_vslot); sig(t % c->mail_ring); sig(k == K ? tau_b % c->label_ring : 0);
    if (enqueue) {
      T* gin = reinterpret_cast<T*>(m.temps[0]);
      if (k < K) {
        // receive + shrink (Eq. 15): the mailbox of module k+1 holds the gradient it produced at t-1
        const Module& dn = c->mods[k];
        const T* recv = reinterpret_cast<const T*>(dn.mail) + (size_t)((t - 1) % c->mail_ring) * align_up(dn.in_elems, 128);
        scale_tensor<T>(L, recv, gin, c->cfg.beta, dn.in_elems);
      } else {
        head_forward_backward<T>(c, m, L, tau_b, slot, vslot, gin);
        if (loss_dev && mode != RUN_CAPTURE) L.note(cudaMemcpyAsync(loss_dev, m.loss, sizeof(float), cudaMemcpyDeviceToDevice, st));
      }
      T* gfirst = k >= 2 ? reinterpret_cast<T*>(m.mail) + (size_t)(t % c->mail_ring) * align_up(m.in_elems, 128) : nullptr;
      const bool forked = (mode == RUN_STREAMS || mode == RUN_CAPTURE) && c->cfg.serial == 0;
      Launch LS{c, forked ? m.stream2 : st};
      backward_module<T>(c, m, L, LS, forked, tau_b, slot, vslot, gin, gfirst);
      if (L.err == cudaSuccess) L.err = LS.err;
      update_module<T>(c, m, L, next_vslot);
    }
    m.updates += 1;
    row.tau_b = tau_b; row.ver_b = ver; row.slot_b = slot;
    if (k >= 2) { m.last_grad_batch = tau_b; m.last_grad_slot = (int)(t % c->mail_ring); }
  };
  auto rec = [&](cudaEvent_t e) { if (events) L.note(cudaEventRecord(e, st)); };
  // while the profiler is on, each pass of the module is bracketed by two timing events (after its waits)
  auto pass_mark = [&]() {
    if (!c->profiling || !enqueue || c->mod_event_owner.size() >= kProfMaxPairs) return;
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return;
    c->mod_events.push_back(e);
    if (c->mod_events.size() % 2 == 0) c->mod_event_owner.push_back(k - 1);
    cudaEventRecord(e, st);
  };

  if (k == K) {
    wait_act();
    pass_mark(); do_forward(); pass_mark();
    rec(m.ev_act[e_now]);
    pass_mark(); do_backward_update(); pass_mark();
    rec(m.ev_grad[e_now]);
  } else if (c->cfg.order == FDG_BACKWARD_FIRST) {
    wait_grad();
    pass_mark(); do_backward_update(); pass_mark();
    rec(m.ev_grad[e_now]);
    wait_act();
    pass_mark(); do_forward(); pass_mark();
    rec(m.ev_act[e_now]);
  } else {
    wait_act();
    pass_mark(); do_forward(); pass_mark();
    rec(m.ev_act[e_now]);
    wait_grad();
    pass_mark(); do_backward_update(); pass_mark();
    rec(m.ev_grad[e_now]);
  }
  if (c->log.size() >= kLogIterations * (size_t)K) c->log.erase(c->log.begin(), c->log.begin() + K);
  c->log.push_back(row);
  return L.err;
}

static fdg_status fail(const fdg_ctx* c, fdg_status s, const std::string& msg) {
  if (c) c->err = msg;
  return s;
}
static fdg_status cuda_fail(fdg_ctx* c, cudaError_t e, const char* where) {
  c->latched = FDG_ERR_CUDA;
  return fail(c, FDG_ERR_CUDA, std::string(where) + ": " + cudaGetErrorString(e));
}

static cudaError_t drain(fdg_ctx* c) {
  cudaError_t e = cudaSuccess;
  if (c->stepped) e = cudaStreamSynchronize(c->last_stream);
  for (Module& m : c->mods) {
    cudaError_t r = cudaStreamSynchronize(m.stream);
    if (e == cudaSuccess) e = r;
    if (m.stream2) { r = cudaStreamSynchronize(m.stream2); if (e == cudaSuccess) e = r; }
  }
  return e;
}

}  // namespace fdg

// =================================================================== C ABI ====
extern "C" {

const char* fdg_status_string(fdg_status s) {
  switch (s) {
    case FDG_OK: return "ok";
    case FDG_ERR_INVALID_ARG: return "invalid argument";
    case FDG_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case FDG_ERR_CUDA: return "CUDA error";
    case FDG_ERR_STATE: return "call not valid in this state";
    case FDG_ERR_UNSUPPORTED: return "unsupported configuration";
    case FDG_ERR_NONFINITE: return "non-finite loss";
    case FDG_ERR_TIMEOUT: return "timeout";
  }
  return "unknown status";
}

const char* fdg_last_error(const fdg_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

static fdg_status make_plan(const fdg_arch* arch, const fdg_config* cfg, fdg_ctx* c) {
  std::string why;
  fdg_status s = validate(arch, cfg, &why);
  if (s != FDG_OK) { c->err = why; return s; }
  c->arch = *arch; c->cfg = *cfg; c->K = cfg->K;
  c->splits.assign(cfg->split_after_block, cfg->split_after_block + (cfg->K - 1));
  c->cfg.split_after_block = nullptr;
  c->bf16_mode = cfg->precision == FDG_BF16_TC;
  c->esize = c->bf16_mode ? 2 : 4;
  c->lr = cfg->lr;
  c->use_graphs = cfg->graphs != 0;
  c->period = 1;
  plan_modules(c);
  return FDG_OK;
}

fdg_status fdg_workspace_bytes(const fdg_arch* arch, const fdg_config* cfg, size_t* out_bytes) {
  if (!out_bytes) return FDG_ERR_INVALID_ARG;
  fdg_ctx tmp;
  fdg_status s = make_plan(arch, cfg, &tmp);
  if (s != FDG_OK) return s;
  *out_bytes = carve(&tmp, nullptr);
  return FDG_OK;
}

fdg_status fdg_create(const fdg_arch* arch, const fdg_config* cfg, void* dev_workspace, size_t bytes,
                      const fdg_stream* streams, fdg_ctx** out_ctx) {
  if (!out_ctx) return FDG_ERR_INVALID_ARG;
  *out_ctx = nullptr;
  if (!dev_workspace || (reinterpret_cast<uintptr_t>(dev_workspace) & 255)) return FDG_ERR_INVALID_ARG;
  fdg_ctx* c = new (std::nothrow) fdg_ctx();
  if (!c) return FDG_ERR_STATE;
  fdg_status s = make_plan(arch, cfg, c);
  if (s != FDG_OK) { delete c; return s; }
  const size_t need = carve(c, nullptr);
  if (bytes < need) { delete c; return FDG_ERR_WORKSPACE_TOO_SMALL; }
  cudaError_t e = cudaGetDevice(&c->device);
  if (e == cudaSuccess) e = cudaMemset(dev_workspace, 0, need);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { delete c; return FDG_ERR_CUDA; }
  carve(c, static_cast<char*>(dev_workspace));
  c->ws_base = static_cast<char*>(dev_workspace);
  c->ws_bytes = need;
  {
    std::vector<unsigned long long> table(c->guard_offsets.begin(), c->guard_offsets.end());
    e = cudaMemcpy(c->guard_table, table.data(), table.size() * sizeof(unsigned long long), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) {
      guard_fill_kernel<<<(unsigned)table.size(), (unsigned)(kGuardBytes / 4)>>>(c->ws_base, c->guard_table);
      e = cudaGetLastError();
    }
  }
  for (Module& m : c->mods) {
    if (m.flip_table_dev && e == cudaSuccess)
      e = cudaMemcpy(m.flip_table_dev, m.flip_table.data(), m.flip_table.size() * sizeof(tc::FlipEntry), cudaMemcpyHostToDevice);
    if (m.eval_table_dev && e == cudaSuccess)
      e = cudaMemcpy(m.eval_table_dev, m.eval_table.data(), m.eval_table.size() * sizeof(EvalStatEntry), cudaMemcpyHostToDevice);
    if (m.n_running && e == cudaSuccess) {      // running mean 0 (the cleared workspace), running variance 1
      std::vector<float> init(m.n_running, 0.f);
      for (const EvalStatEntry& en : m.eval_table)
        for (int ch = 0; ch < en.C; ++ch) init[en.roff + en.C + ch] = 1.f;
      e = cudaMemcpy(m.running, init.data(), m.n_running * 4, cudaMemcpyHostToDevice);
    }
  }
  // shared-memory limits of the tensor-core kernels, raised here so that a kernel's first launch may be a recorded one
  if (e == cudaSuccess && c->bf16_mode) e = halo::set_smem_attrs();
  if (e == cudaSuccess && c->bf16_mode) e = tc::conv_tc_set_attrs();
  c->own_streams = streams == nullptr;
  for (int k = 0; k < c->K && e == cudaSuccess; ++k) {
    Module& m = c->mods[k];
    if (streams) m.stream = static_cast<cudaStream_t>(streams[k]);
    else e = cudaStreamCreateWithFlags(&m.stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&m.stream2, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m.ev_fork2, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m.ev_join2, cudaEventDisableTiming);
    for (int i = 0; i < 4 && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&m.ev_buf[i], cudaEventDisableTiming);
    for (int i = 0; i < kEventRing && e == cudaSuccess; ++i) {
      e = cudaEventCreateWithFlags(&m.ev_act[i], cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m.ev_grad[i], cudaEventDisableTiming);
    }
  }
  for (int i = 0; i < kEventRing && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&c->ev_in[i], cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_staged, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_ingested, cudaEventDisableTiming);
  if (e == cudaSuccess && c->use_graphs) e = cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking);
  c->ev_cjoin.assign(c->K, nullptr);
  for (int k = 0; k < c->K && e == cudaSuccess; ++k) e = cudaEventCreateWithFlags(&c->ev_cjoin[k], cudaEventDisableTiming);
  // Convolution launches are sized for the module streams running side by side: 148 / K SMs each.  With 128
  // image tiles per layer that is 2 tiles per CTA at K = 2 and 4 at K = 4 (32 CTAs; measured against 3, 5, 6 and
  // 8 tiles per CTA: the four chains' convolutions then fit the SMs together and a CTA's start-up is paid once
  // per four tiles).
  c->tmaps.share = c->cfg.serial ? 1 : c->K;
  c->tmaps.wgrad_side_cap = 16;
  // Blocks of a batch-norm apply kernel that first re-adds a convolution's partial sums: 4 per SM shared
  // between the module streams, not fewer than 222 (measured: 222 blocks at K = 4 against 74 / 111 / 148 / 185 /
  // 259 / 296; K = 2 is flat between 222 and 592).
  c->ew_block_cap = c->cfg.serial ? 4 * 148 : std::max(222, 4 * 148 / c->K);
  c->graph_exec.assign(c->period, nullptr);
  c->graph_sig.assign(c->period, 0);
  c->graph_launches.assign(c->period, 0);
  // The clearing of the workspace and the table uploads above ran on the default stream, which the module
  // streams (non-blocking) do not wait for: nothing may be enqueued on them before those have finished.
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { delete c; return FDG_ERR_CUDA; }
  *out_ctx = c;
  return FDG_OK;
}

fdg_status fdg_destroy(fdg_ctx* c) {
  if (!c) return FDG_ERR_INVALID_ARG;
  cudaError_t e = drain(c);
  for (Module& m : c->mods) {
    for (int i = 0; i < kEventRing; ++i) { cudaEventDestroy(m.ev_act[i]); cudaEventDestroy(m.ev_grad[i]); }
    if (c->own_streams && m.stream) cudaStreamDestroy(m.stream);
    if (m.stream2) cudaStreamDestroy(m.stream2);
    if (m.ev_fork2) cudaEventDestroy(m.ev_fork2);
    if (m.ev_join2) cudaEventDestroy(m.ev_join2);
    for (int i = 0; i < 4; ++i) if (m.ev_buf[i]) cudaEventDestroy(m.ev_buf[i]);
  }
  for (int i = 0; i < kEventRing; ++i) cudaEventDestroy(c->ev_in[i]);
  cudaEventDestroy(c->ev_join);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_staged) cudaEventDestroy(c->ev_staged);
  if (c->ev_ingested) cudaEventDestroy(c->ev_ingested);
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
  for (cudaEvent_t ev : c->ev_cjoin) if (ev) cudaEventDestroy(ev);
  for (cudaGraphExec_t g : c->graph_exec) if (g) cudaGraphExecDestroy(g);
  for (cudaEvent_t ev : c->prof_events) cudaEventDestroy(ev);
  for (cudaEvent_t ev : c->mod_events) cudaEventDestroy(ev);
  delete c;
  return e == cudaSuccess ? FDG_OK : FDG_ERR_CUDA;
}

#define FDG_MODULE_OR_FAIL(c, module)                                        \
  if (!(c)) return FDG_ERR_INVALID_ARG;                                      \
  if ((module) < 1 || (module) > (c)->K) return fail((c), FDG_ERR_INVALID_ARG, "module index out of range")

fdg_status fdg_param_count(const fdg_ctx* c, int module, size_t* out_n) {
  FDG_MODULE_OR_FAIL(c, module);
  if (!out_n) return FDG_ERR_INVALID_ARG;
  *out_n = c->mods[module - 1].n_params;
  return FDG_OK;
}

fdg_status fdg_param_layout(const fdg_ctx* c, int module, fdg_param_entry* dst, size_t cap, size_t* out_n) {
  FDG_MODULE_OR_FAIL(c, module);
  const auto& lay = c->mods[module - 1].layout;
  if (out_n) *out_n = lay.size();
  if (dst) for (size_t i = 0; i < std::min(cap, lay.size()); ++i) dst[i] = lay[i];
  return FDG_OK;
}

static fdg_status copy_vec(fdg_ctx* c, int module, float* dev_vec, const float* src, float* dst, size_t n, bool refresh) {
  FDG_MODULE_OR_FAIL(c, module);
  Module& m = c->mods[module - 1];
  if (n != m.n_params || (!src && !dst)) return fail(c, FDG_ERR_INVALID_ARG, "element count does not match fdg_param_count");
  cudaError_t e = drain(c);
  if (e == cudaSuccess && n) {
    if (src) e = cudaMemcpy(dev_vec, src, n * 4, cudaMemcpyDefault);
    else e = cudaMemcpy(dst, dev_vec, n * 4, cudaMemcpyDefault);
    // A copy from pageable host memory returns when the data is staged, not when it has reached the device,
    // and the module streams (non-blocking) do not wait for the default stream the copy runs on: everything
    // below, and every later kernel that reads this vector, has to start after the copy has landed.
    if (e == cudaSuccess && src) e = cudaDeviceSynchronize();
  }
  if (e == cudaSuccess && refresh && n) {
    for (int v = 0; v < m.Dw && e == cudaSuccess; ++v) {
      e = cudaMemcpyAsync(m.wver + (size_t)v * align_up(n, 64), m.theta, n * 4, cudaMemcpyDeviceToDevice, m.stream);
      if (e == cudaSuccess && c->bf16_mode) {
        cast_kernel<bf16><<<(int)std::min<size_t>((n + 255) / 256, 1184), 256, 0, m.stream>>>(m.theta, m.wver16 + (size_t)v * align_up(n, 64), n);
        ++c->launches;
        e = cudaGetLastError();
        if (e == cudaSuccess && m.flip_table_dev) {
          tc::wflip_kernel<<<dim3(m.flip_blocks, (unsigned)m.flip_table.size()), 256, 0, m.stream>>>(
              m.wver16 + (size_t)v * align_up(n, 64), m.wflip16 + (size_t)v * m.flip_elems, m.flip_table_dev);
          ++c->launches;
          e = cudaGetLastError();
        }
      }
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(m.stream);
  }
  return e == cudaSuccess ? FDG_OK : cuda_fail(c, e, "parameter copy");
}

fdg_status fdg_set_params(fdg_ctx* c, int module, const float* src, size_t n) {
  if (!src) return FDG_ERR_INVALID_ARG;
  FDG_MODULE_OR_FAIL(c, module);
  return copy_vec(c, module, c->mods[module - 1].theta, src, nullptr, n, true);
}
fdg_status fdg_set_momentum(fdg_ctx* c, int module, const float* src, size_t n) {
  if (!src) return FDG_ERR_INVALID_ARG;
  FDG_MODULE_OR_FAIL(c, module);
  return copy_vec(c, module, c->mods[module - 1].mom, src, nullptr, n, false);
}
fdg_status fdg_get_params(fdg_ctx* c, int module, float* dst, size_t n) {
  if (!dst) return FDG_ERR_INVALID_ARG;
  FDG_MODULE_OR_FAIL(c, module);
  return copy_vec(c, module, c->mods[module - 1].theta, nullptr, dst, n, false);
}
fdg_status fdg_get_grads(fdg_ctx* c, int module, float* dst, size_t n) {
  if (!dst) return FDG_ERR_INVALID_ARG;
  FDG_MODULE_OR_FAIL(c, module);
  return copy_vec(c, module, c->mods[module - 1].grad, nullptr, dst, n, false);
}
fdg_status fdg_get_momentum(fdg_ctx* c, int module, float* dst, size_t n) {
  if (!dst) return FDG_ERR_INVALID_ARG;
  FDG_MODULE_OR_FAIL(c, module);
  return copy_vec(c, module, c->mods[module - 1].mom, nullptr, dst, n, false);
}

fdg_status fdg_set_lr(fdg_ctx* c, float lr) {
  if (!c) return FDG_ERR_INVALID_ARG;
  if (!(lr >= 0.f)) return fail(c, FDG_ERR_INVALID_ARG, "learning rate must be >= 0");
  c->lr = lr;
  return FDG_OK;
}

// Host-side state of the modules that a dry run advances (restored if a recorded graph turns out stale).
struct HostState {
  std::vector<int64_t> updates, last_out_batch, last_grad_batch;
  std::vector<int> last_out_slot, last_grad_slot;
  std::vector<std::vector<int64_t>> slot_version, slot_batch;
  size_t log_size;
};
static HostState save_host_state(const fdg_ctx* c) {
  HostState h;
  for (const Module& m : c->mods) {
    h.updates.push_back(m.updates); h.last_out_batch.push_back(m.last_out_batch); h.last_grad_batch.push_back(m.last_grad_batch);
    h.last_out_slot.push_back(m.last_out_slot); h.last_grad_slot.push_back(m.last_grad_slot);
    h.slot_version.push_back(m.slot_version); h.slot_batch.push_back(m.slot_batch);
  }
  h.log_size = c->log.size();
  return h;
}
static void restore_host_state(fdg_ctx* c, const HostState& h) {
  for (size_t i = 0; i < c->mods.size(); ++i) {
    Module& m = c->mods[i];
    m.updates = h.updates[i]; m.last_out_batch = h.last_out_batch[i]; m.last_grad_batch = h.last_grad_batch[i];
    m.last_out_slot = h.last_out_slot[i]; m.last_grad_slot = h.last_grad_slot[i];
    m.slot_version = h.slot_version[i]; m.slot_batch = h.slot_batch[i];
  }
  if (c->log.size() > h.log_size) c->log.resize(h.log_size);
}

static cudaError_t run_modules(fdg_ctx* c, cudaStream_t cs, StepMode mode, float* loss_dev) {
  c->step_sig = 0;
  for (int k = 0; k < c->K; ++k) {
    Module& m = c->mods[k];
    const bool one_stream = mode == RUN_SERIAL || c->cfg.serial != 0;
    cudaStream_t st = one_stream ? cs : m.stream;
    cudaError_t e = cudaSuccess;
    if (mode == RUN_CAPTURE && !one_stream) e = cudaStreamWaitEvent(st, c->ev_fork, 0);   // the module's stream joins the recording
    if (e == cudaSuccess)
      e = c->bf16_mode ? module_step<bf16>(c, m, st, mode, loss_dev) : module_step<float>(c, m, st, mode, loss_dev);
    if (e == cudaSuccess && mode == RUN_CAPTURE && !one_stream) {
      e = cudaEventRecord(c->ev_cjoin[k], st);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(cs, c->ev_cjoin[k], 0);
    }
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// One iteration through a CUDA graph: replay the graph recorded for this phase of the rings, or
// record it now.  The ingest and the learning rate stay outside the graph (they depend on the call).
static cudaError_t graph_step(fdg_ctx* c, cudaStream_t cs, float* loss_dev) {
  const int phase = (int)(c->t % c->period);
  cudaError_t e = cudaSuccess;
  if (c->lr_on_device != c->lr) {
    set_scalar_kernel<<<1, 1, 0, cs>>>(c->lr_dev, c->lr);
    ++c->launches;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    c->lr_on_device = c->lr;
  }
  if (c->graph_exec[phase]) {
    const HostState saved = save_host_state(c);
    e = run_modules(c, cs, RUN_DRY, nullptr);
    if (e != cudaSuccess) return e;
    if (c->step_sig == c->graph_sig[phase]) {
      c->launches += c->graph_launches[phase];
      e = cudaGraphLaunch(c->graph_exec[phase], cs);
    } else {                               // the slots moved: record again
      restore_host_state(c, saved);
      cudaGraphExecDestroy(c->graph_exec[phase]);
      c->graph_exec[phase] = nullptr;
    }
  }
  if (!c->graph_exec[phase]) {
    const uint64_t l0 = c->launches;
    e = cudaStreamBeginCapture(c->cap_stream, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) return e;
    e = cudaEventRecord(c->ev_fork, c->cap_stream);
    if (e == cudaSuccess) e = run_modules(c, c->cap_stream, RUN_CAPTURE, nullptr);
    cudaGraph_t graph = nullptr;
    cudaError_t e2 = cudaStreamEndCapture(c->cap_stream, &graph);
    if (e == cudaSuccess) e = e2;
    if (e == cudaSuccess) e = cudaGraphInstantiate(&c->graph_exec[phase], graph, 0);
    if (graph) cudaGraphDestroy(graph);
    if (e != cudaSuccess) { c->graph_exec[phase] = nullptr; return e; }
    c->graph_sig[phase] = c->step_sig;
    c->graph_launches[phase] = c->launches - l0;
    e = cudaGraphLaunch(c->graph_exec[phase], cs);
  }
  if (e == cudaSuccess && loss_dev && c->t >= c->K)
    e = cudaMemcpyAsync(loss_dev, c->mods[c->K - 1].loss, sizeof(float), cudaMemcpyDeviceToDevice, cs);
  return e;
}

fdg_status fdg_step(fdg_ctx* c, fdg_stream stream, const float* images_dev, const int32_t* labels_dev, float* loss_dev) {
  if (!c) return FDG_ERR_INVALID_ARG;
  if (!images_dev || !labels_dev) return fail(c, FDG_ERR_INVALID_ARG, "images and labels must not be null");
  if (c->latched != FDG_OK) return c->latched;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const bool serial = c->cfg.serial != 0;
  c->last_stream = cs; c->stepped = true;
  c->t += 1;
  const int64_t t = c->t;
  if (c->has_schedule) fdg_lr_at(&c->schedule, t, &c->lr);
  Module& m1 = c->mods[0];
  cudaError_t e = cudaSuccess;
  // Graphs take over once every module has run each of its passes at least once (all kernels
  // have been launched the ordinary way, their attributes are set, the pipeline is full).
  if (c->use_graphs && !c->graph_mode_entered && t > 2 * (int64_t)c->K + 1) {
    for (Module& m : c->mods) {              // from here on every iteration is ordered on the caller's stream
      if (e == cudaSuccess) e = cudaEventRecord(c->ev_join, m.stream);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(cs, c->ev_join, 0);
    }
    if (e != cudaSuccess) return cuda_fail(c, e, "entering graph mode");
    c->graph_mode_entered = true;
  }
  const bool graph = c->graph_mode_entered;
  // a0: ingest batch t into module 1's image ring and the label ring
  if (!serial && !graph) e = cudaStreamWaitEvent(cs, m1.ev_grad[(t - 1) % kEventRing], 0);
  if (e != cudaSuccess) return cuda_fail(c, e, "ingest wait");
  {
    const size_t rows = (size_t)c->arch.batch * c->arch.in_h * c->arch.in_w;
    int32_t* lab = c->labels + (size_t)(t % c->label_ring) * c->arch.batch;
    const size_t slot_off = (size_t)(t % m1.Din) * align_up(m1.in_elems, 128);
    Launch L{c, cs};
    L.begin(KC_INGEST, (double)rows * (c->arch.in_c * 4 + m1.in_c * c->esize), 0.0);
    if (c->bf16_mode)
      L.note(launch_ingest<bf16>(cs, images_dev, reinterpret_cast<bf16*>(m1.in_ring) + slot_off, rows, c->arch.in_c, m1.in_c, labels_dev, lab, c->arch.batch));
    else
      L.note(launch_ingest<float>(cs, images_dev, reinterpret_cast<float*>(m1.in_ring) + slot_off, rows, c->arch.in_c, m1.in_c, labels_dev, lab, c->arch.batch));
    ++c->launches;
    e = L.err;
    if (e == cudaSuccess && !serial && !graph) e = cudaEventRecord(c->ev_in[t % kEventRing], cs);
    if (e == cudaSuccess && c->record_ingested) e = cudaEventRecord(c->ev_ingested, cs);
    if (e != cudaSuccess) return cuda_fail(c, e, "ingest");
  }
  if (graph) e = graph_step(c, cs, loss_dev);
  else e = run_modules(c, cs, serial ? RUN_SERIAL : RUN_STREAMS, loss_dev);
  if (e != cudaSuccess) return cuda_fail(c, e, "module step");
  return FDG_OK;
}

fdg_status fdg_step_host(fdg_ctx* c, fdg_stream stream, const float* images_host, const int32_t* labels_host,
                         float* loss_host) {
  if (!c) return FDG_ERR_INVALID_ARG;
  if (!images_host || !labels_host) return fail(c, FDG_ERR_INVALID_ARG, "images and labels must not be null");
  if (c->latched != FDG_OK) return c->latched;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const size_t img_bytes = (size_t)c->arch.batch * c->arch.in_h * c->arch.in_w * c->arch.in_c * 4;
  // The copy waits only for the ingest of the call before (which read the staging buffers), not for that call's
  // module-steps: from pinned memory it runs beside them.  (An event that was never recorded does not block.)
  cudaError_t e = cudaStreamWaitEvent(c->copy_stream, c->ev_ingested, 0);
  if (e == cudaSuccess) e = cudaMemcpyAsync(c->host_images, images_host, img_bytes, cudaMemcpyHostToDevice, c->copy_stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(c->host_labels, labels_host, (size_t)c->arch.batch * 4, cudaMemcpyHostToDevice, c->copy_stream);
  if (e == cudaSuccess) e = cudaEventRecord(c->ev_staged, c->copy_stream);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(cs, c->ev_staged, 0);
  if (e != cudaSuccess) return cuda_fail(c, e, "host to device copy");
  c->record_ingested = true;
  fdg_status s = fdg_step(c, stream, c->host_images, c->host_labels, nullptr);
  c->record_ingested = false;
  if (s != FDG_OK) return s;
  if (loss_host && c->t >= c->K) {
    Module& mk = c->mods[c->K - 1];
    e = cudaMemcpyAsync(loss_host, mk.loss, sizeof(float), cudaMemcpyDeviceToHost,
                        (c->cfg.serial || c->graph_mode_entered) ? cs : mk.stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "loss copy");
  }
  return FDG_OK;
}

fdg_status fdg_sync(fdg_ctx* c, fdg_stream stream) {
  if (!c) return FDG_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaSuccess;
  if (!c->cfg.serial)
    for (Module& m : c->mods) {
      if (e == cudaSuccess) e = cudaEventRecord(c->ev_join, m.stream);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(cs, c->ev_join, 0);
    }
  if (e == cudaSuccess) e = cudaStreamSynchronize(cs);
  int flags[3] = {0, 0, 0};
  if (e == cudaSuccess) e = cudaMemcpy(flags, c->flags, sizeof(flags), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(c, e, "sync");
  if (flags[0] || flags[1] || flags[2]) {
    cudaMemset(c->flags, 0, sizeof(flags));
    if (flags[2]) { c->latched = FDG_ERR_TIMEOUT; return fail(c, FDG_ERR_TIMEOUT, "a tensor-core kernel gave up waiting on a barrier"); }
    if (flags[1]) return fail(c, FDG_ERR_INVALID_ARG, "a label was outside [0, num_classes)");
    return fail(c, FDG_ERR_NONFINITE, "a loss computed since the last sync was NaN or Inf");
  }
  return c->latched;
}

fdg_status fdg_debug_raise_flag(fdg_ctx* c, int which) {
  if (!c) return FDG_ERR_INVALID_ARG;
  if (which < 0 || which > 2) return fail(c, FDG_ERR_INVALID_ARG, "no such status word");
  cudaError_t e = drain(c);
  const int one = 1;
  if (e == cudaSuccess) e = cudaMemcpy(c->flags + which, &one, sizeof(int), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  return e == cudaSuccess ? FDG_OK : cuda_fail(c, e, "raising a status word");
}

fdg_status fdg_debug_guard_count(const fdg_ctx* c, size_t* out_count) {
  if (!c || !out_count) return FDG_ERR_INVALID_ARG;
  *out_count = c->guard_offsets.size();
  return FDG_OK;
}

fdg_status fdg_debug_guard_offset(const fdg_ctx* c, size_t index, size_t* out_byte_offset) {
  if (!c || !out_byte_offset || index >= c->guard_offsets.size()) return FDG_ERR_INVALID_ARG;
  *out_byte_offset = c->guard_offsets[index];
  return FDG_OK;
}

fdg_status fdg_debug_check_guards(fdg_ctx* c, long long* out_first_bad) {
  if (!c || !out_first_bad) return FDG_ERR_INVALID_ARG;
  cudaError_t e = drain(c);
  const int none = INT_MAX;
  if (e == cudaSuccess) e = cudaMemcpy(c->flags + 3, &none, sizeof(int), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) {
    guard_check_kernel<<<(unsigned)c->guard_offsets.size(), (unsigned)(kGuardBytes / 4)>>>(c->ws_base, c->guard_table, c->flags + 3);
    ++c->launches;
    e = cudaGetLastError();
  }
  int got = none;
  if (e == cudaSuccess) e = cudaMemcpy(&got, c->flags + 3, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(c, e, "guard check");
  *out_first_bad = got == none ? -1 : (long long)got;
  return FDG_OK;
}

fdg_status fdg_debug_wait_probe(fdg_ctx* c, fdg_stream stream, unsigned poll_limit) {
  if (!c) return FDG_ERR_INVALID_ARG;
  if (poll_limit < 1 || poll_limit > (1u << 20)) return fail(c, FDG_ERR_INVALID_ARG, "poll limit outside 1..2^20");
  tc::wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(poll_limit, c->flags + 2);
  ++c->launches;
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? FDG_OK : cuda_fail(c, e, "wait probe");
}

static fdg_status export_tensor(fdg_ctx* c, const void* src, size_t rows, int c_store, int c_logical, float* dst, size_t n) {
  if (n != rows * (size_t)c_logical) return fail(c, FDG_ERR_INVALID_ARG, "element count does not match fdg_boundary_elems");
  cudaError_t e = drain(c);
  if (e != cudaSuccess) return cuda_fail(c, e, "drain");
  const int blocks = ew_blocks(n);
  if (c->bf16_mode) export_kernel<bf16><<<blocks, 256>>>(static_cast<const bf16*>(src), c->staging, rows, c_store, c_logical);
  else export_kernel<float><<<blocks, 256>>>(static_cast<const float*>(src), c->staging, rows, c_store, c_logical);
  ++c->launches;
  e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaMemcpy(dst, c->staging, n * 4, cudaMemcpyDefault);
  return e == cudaSuccess ? FDG_OK : cuda_fail(c, e, "export");
}

fdg_status fdg_lr_at(const fdg_lr_schedule* s, int64_t iteration, float* out_lr) {
  if (!s || !out_lr || iteration < 1 || s->iters_per_epoch < 1 || s->n_milestones < 0 || s->n_milestones > 8 ||
      !(s->base_lr >= 0.f) || !(s->gamma >= 0.f) || s->warmup_epochs < 0 || !(s->warmup_lr >= 0.f)) return FDG_ERR_INVALID_ARG;
  const int64_t epoch = (iteration - 1) / s->iters_per_epoch;
  if (epoch < s->warmup_epochs) { *out_lr = s->warmup_lr; return FDG_OK; }
  double lr = s->base_lr;
  for (int i = 0; i < s->n_milestones; ++i) if (epoch >= s->milestones[i]) lr *= s->gamma;
  *out_lr = (float)lr;
  return FDG_OK;
}

fdg_status fdg_set_lr_schedule(fdg_ctx* c, const fdg_lr_schedule* s) {
  if (!c) return FDG_ERR_INVALID_ARG;
  if (!s) { c->has_schedule = false; return FDG_OK; }
  float probe;
  if (fdg_lr_at(s, 1, &probe) != FDG_OK) return fail(c, FDG_ERR_INVALID_ARG, "bad learning-rate schedule");
  c->schedule = *s;
  c->has_schedule = true;
  return FDG_OK;
}

fdg_status fdg_bn_running_count(const fdg_ctx* c, int module, size_t* out_n) {
  FDG_MODULE_OR_FAIL(c, module);
  if (!out_n) return FDG_ERR_INVALID_ARG;
  *out_n = c->mods[module - 1].n_running;
  return FDG_OK;
}
static fdg_status copy_running(fdg_ctx* c, int module, const float* src, float* dst, size_t n) {
  FDG_MODULE_OR_FAIL(c, module);
  Module& m = c->mods[module - 1];
  if (n != m.n_running || (!src && !dst)) return fail(c, FDG_ERR_INVALID_ARG, "element count does not match fdg_bn_running_count");
  cudaError_t e = drain(c);
  if (e == cudaSuccess && n) e = src ? cudaMemcpy(m.running, src, n * 4, cudaMemcpyDefault) : cudaMemcpy(dst, m.running, n * 4, cudaMemcpyDefault);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  return e == cudaSuccess ? FDG_OK : cuda_fail(c, e, "running statistics copy");
}
fdg_status fdg_get_bn_running(fdg_ctx* c, int module, float* dst, size_t n) { return dst ? copy_running(c, module, nullptr, dst, n) : FDG_ERR_INVALID_ARG; }
fdg_status fdg_set_bn_running(fdg_ctx* c, int module, const float* src, size_t n) { return src ? copy_running(c, module, src, nullptr, n) : FDG_ERR_INVALID_ARG; }

}  // extern "C"

template <typename T>
static cudaError_t eval_all(fdg_ctx* c, cudaStream_t cs, const float* images_dev, const int32_t* labels_dev, float* logits_dev,
                            int* correct_dev) {
  Module& m1 = c->mods[0];
  const size_t rows = (size_t)c->arch.batch * c->arch.in_h * c->arch.in_w;
  Launch L{c, cs};
  L.begin(KC_INGEST, (double)rows * (c->arch.in_c * 4 + m1.in_c * c->esize), 0.0);
  L.note(launch_ingest<T>(cs, images_dev, reinterpret_cast<T*>(m1.in_ring) + (size_t)m1.Din * align_up(m1.in_elems, 128), rows,
                          c->arch.in_c, m1.in_c, nullptr, nullptr, 0));
  ++c->launches;
  for (Module& m : c->mods) {
    const int vslot = (int)(m.updates % m.Dw);
    if (m.eval_table_dev) {
      bn_eval_stats_kernel<<<(unsigned)m.eval_table.size(), 128, 0, cs>>>(m.running, slot_F(m, m.D), m.eval_table_dev, c->arch.bn_eps);
      L.check();
    }
    forward_module<T>(c, m, L, 0, m.D, vslot, true);
    if (m.k == c->K) head_eval<T>(c, m, L, m.D, vslot, labels_dev, logits_dev, correct_dev);
  }
  return L.err;
}

extern "C" {

fdg_status fdg_eval(fdg_ctx* c, fdg_stream stream, const float* images_dev, const int32_t* labels_dev, float* logits_dev,
                    int* correct_dev) {
  if (!c) return FDG_ERR_INVALID_ARG;
  if (!images_dev || (correct_dev && !labels_dev)) return fail(c, FDG_ERR_INVALID_ARG, "images (and labels, to count) must not be null");
  if (c->latched != FDG_OK) return c->latched;
  cudaError_t e = drain(c);
  if (e != cudaSuccess) return cuda_fail(c, e, "drain");
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int share = c->tmaps.share;
  c->tmaps.share = 1;                    // the pass runs alone: a launch may take every SM
  e = c->bf16_mode ? eval_all<bf16>(c, cs, images_dev, labels_dev, logits_dev, correct_dev)
                   : eval_all<float>(c, cs, images_dev, labels_dev, logits_dev, correct_dev);
  c->tmaps.share = share;
  c->last_stream = cs; c->stepped = true;
  return e == cudaSuccess ? FDG_OK : cuda_fail(c, e, "inference pass");
}

fdg_status fdg_drain(fdg_ctx* c, fdg_stream stream, float* losses_dev) {
  if (!c) return FDG_ERR_INVALID_ARG;
  if (c->latched != FDG_OK) return c->latched;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  cudaError_t e = drain(c);
  if (e != cudaSuccess) return cuda_fail(c, e, "drain");
  if (c->t > 0) {
    // From here on the iterations are issued the ordinary way (a recorded graph holds passes that must now be
    // skipped); the host has waited for everything, so stream order is all that is needed.
    c->graph_mode_entered = false;
    c->last_batch = c->t;
    c->last_stream = cs; c->stepped = true;
    for (int i = 0; i < 2 * c->K - 2 && e == cudaSuccess; ++i) {
      c->t += 1;
      if (c->has_schedule) fdg_lr_at(&c->schedule, c->t, &c->lr);
      e = run_modules(c, cs, c->cfg.serial ? RUN_SERIAL : RUN_STREAMS, losses_dev ? losses_dev + i : nullptr);
    }
    c->last_batch = INT64_MAX;
    if (e != cudaSuccess) return cuda_fail(c, e, "draining iterations");
    e = drain(c);
    if (e != cudaSuccess) return cuda_fail(c, e, "drain");
  }
  c->t = 0;
  for (Module& m : c->mods) {
    std::fill(m.slot_version.begin(), m.slot_version.end(), -1);
    std::fill(m.slot_batch.begin(), m.slot_batch.end(), -1);
    m.last_out_batch = m.last_grad_batch = -1;
    m.last_out_slot = m.last_grad_slot = -1;
  }
  return FDG_OK;
}

// Host-side part of a saved state: a fixed header, then per module its counters and slot tables.
struct StateHeader {
  uint64_t magic, ws_bytes;
  int64_t t;
  float lr;
  int32_t K, period, graph_mode_entered;
};
constexpr uint64_t kStateMagic = 0x4644475354415445ull;      // "FDGSTATE"
static size_t state_host_bytes(const fdg_ctx* c) {
  size_t n = sizeof(StateHeader);
  for (const Module& m : c->mods) n += (5 + 2 * (size_t)m.D) * sizeof(int64_t);
  return align_up(n, 256);
}

fdg_status fdg_state_bytes(const fdg_ctx* c, size_t* out_bytes) {
  if (!c || !out_bytes) return FDG_ERR_INVALID_ARG;
  *out_bytes = state_host_bytes(c) + c->ws_bytes;
  return FDG_OK;
}

fdg_status fdg_save_state(fdg_ctx* c, void* dst, size_t bytes) {
  if (!c || !dst) return FDG_ERR_INVALID_ARG;
  const size_t hb = state_host_bytes(c);
  if (bytes < hb + c->ws_bytes) return fail(c, FDG_ERR_WORKSPACE_TOO_SMALL, "buffer smaller than fdg_state_bytes");
  cudaError_t e = drain(c);
  if (e != cudaSuccess) return cuda_fail(c, e, "drain");
  std::vector<char> host(hb, 0);
  StateHeader h{kStateMagic, c->ws_bytes, c->t, c->lr, c->K, c->period, c->graph_mode_entered ? 1 : 0};
  std::memcpy(host.data(), &h, sizeof(h));
  int64_t* p = reinterpret_cast<int64_t*>(host.data() + sizeof(StateHeader));
  for (const Module& m : c->mods) {
    *p++ = m.updates; *p++ = m.last_out_batch; *p++ = m.last_grad_batch; *p++ = m.last_out_slot; *p++ = m.last_grad_slot;
    for (int i = 0; i < m.D; ++i) { *p++ = m.slot_version[i]; *p++ = m.slot_batch[i]; }
  }
  e = cudaMemcpy(dst, host.data(), hb, cudaMemcpyDefault);
  if (e == cudaSuccess) e = cudaMemcpy(static_cast<char*>(dst) + hb, c->ws_base, c->ws_bytes, cudaMemcpyDefault);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  return e == cudaSuccess ? FDG_OK : cuda_fail(c, e, "saving the state");
}

fdg_status fdg_load_state(fdg_ctx* c, const void* src, size_t bytes) {
  if (!c || !src) return FDG_ERR_INVALID_ARG;
  const size_t hb = state_host_bytes(c);
  if (bytes < hb + c->ws_bytes) return fail(c, FDG_ERR_INVALID_ARG, "buffer smaller than this context's state");
  cudaError_t e = drain(c);
  if (e != cudaSuccess) return cuda_fail(c, e, "drain");
  std::vector<char> host(hb);
  e = cudaMemcpy(host.data(), src, hb, cudaMemcpyDefault);
  if (e != cudaSuccess) return cuda_fail(c, e, "reading the state");
  StateHeader h;
  std::memcpy(&h, host.data(), sizeof(h));
  if (h.magic != kStateMagic || h.ws_bytes != c->ws_bytes || h.K != c->K || h.period != c->period)
    return fail(c, FDG_ERR_INVALID_ARG, "the state belongs to another architecture or configuration");
  e = cudaMemcpy(c->ws_base, static_cast<const char*>(src) + hb, c->ws_bytes, cudaMemcpyDefault);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { c->latched = FDG_ERR_CUDA; return cuda_fail(c, e, "loading the state"); }
  c->t = h.t; c->lr = h.lr; c->lr_on_device = -1.f;
  c->graph_mode_entered = c->use_graphs && h.graph_mode_entered != 0;
  const int64_t* p = reinterpret_cast<const int64_t*>(host.data() + sizeof(StateHeader));
  for (Module& m : c->mods) {
    m.updates = *p++; m.last_out_batch = *p++; m.last_grad_batch = *p++; m.last_out_slot = (int)*p++; m.last_grad_slot = (int)*p++;
    for (int i = 0; i < m.D; ++i) { m.slot_version[i] = *p++; m.slot_batch[i] = *p++; }
    m.cap_batch = -1;
  }
  c->latched = FDG_OK;
  return FDG_OK;
}

fdg_status fdg_boundary_elems(const fdg_ctx* c, int module, size_t* out_elems, size_t* in_elems) {
  FDG_MODULE_OR_FAIL(c, module);
  const Module& m = c->mods[module - 1];
  if (out_elems) *out_elems = m.out_elems;
  if (in_elems) *in_elems = (size_t)c->arch.batch * m.in_h * m.in_w * m.in_c_logical;
  return FDG_OK;
}

fdg_status fdg_get_module_output(fdg_ctx* c, int module, float* dst, size_t n, int64_t* batch_index) {
  FDG_MODULE_OR_FAIL(c, module);
  if (!dst || !batch_index) return FDG_ERR_INVALID_ARG;
  if (module == c->K) return fail(c, FDG_ERR_INVALID_ARG, "the top module has no output activation");
  Module& m = c->mods[module - 1];
  *batch_index = m.last_out_batch;
  if (m.last_out_batch < 0) return FDG_OK;
  const size_t off = (size_t)m.last_out_slot * m.slot_elems + m.units.back().t_y;
  const char* src = m.fifo + off * c->esize;
  const Unit& u = m.units.back();
  return export_tensor(c, src, (size_t)c->arch.batch * u.P * u.Q, u.co, u.co, dst, n);
}

fdg_status fdg_get_input_grad(fdg_ctx* c, int module, float* dst, size_t n, int64_t* batch_index) {
  FDG_MODULE_OR_FAIL(c, module);
  if (!dst || !batch_index) return FDG_ERR_INVALID_ARG;
  if (module == 1) return fail(c, FDG_ERR_INVALID_ARG, "the gradient with respect to the images is never formed");
  Module& m = c->mods[module - 1];
  *batch_index = m.last_grad_batch;
  if (m.last_grad_batch < 0) return FDG_OK;
  const char* src = m.mail + (size_t)m.last_grad_slot * align_up(m.in_elems, 128) * c->esize;
  return export_tensor(c, src, (size_t)c->arch.batch * m.in_h * m.in_w, m.in_c, m.in_c_logical, dst, n);
}

fdg_status fdg_get_saved_tensor_of(fdg_ctx* c, int module, int unit, int which, int64_t batch, float* dst, size_t n,
                                   size_t* out_elems, int64_t* batch_index) {
  FDG_MODULE_OR_FAIL(c, module);
  Module& m = c->mods[module - 1];
  if (unit < 0 || unit >= (int)m.units.size() || m.units[unit].type == U_HEAD)
    return fail(c, FDG_ERR_INVALID_ARG, "unit index out of range");
  const Unit& u = m.units[unit];
  const size_t B = c->arch.batch;
  const size_t in_e = B * u.H * u.W * u.ci, out_e = B * u.P * u.Q * u.co;
  size_t off = 0, elems = out_e;
  int ch = u.co;
  bool ok = false;
  if (u.type == U_STEM) {
    if (which == 0 && u.bn) { off = u.t_a; ok = true; }
    if (which == 3) { off = u.t_y; ok = true; }
  } else if (u.type == U_BASIC) {
    if (which == 0) { off = u.t_a; ok = true; }
    if (which == 1) { off = u.t_b; ok = true; }
    if (which == 2) { off = u.t_c; ok = true; }
    if (which == 3) { off = u.t_y; ok = true; }
    if (which == 4 && u.proj) { off = u.t_s; ok = true; }
  } else {
    if (which == 0) { off = u.t_a; elems = in_e; ch = u.ci; ok = true; }
    if (which == 1) { off = u.t_b; ok = true; }
    if (which == 2) { off = u.t_c; ok = true; }
    if (which == 3) { off = u.t_y; ok = true; }
  }
  if (!ok) return fail(c, FDG_ERR_INVALID_ARG, "this unit saves no such tensor");
  if (out_elems) *out_elems = elems;
  if (!dst) return FDG_OK;
  if (!batch_index) return FDG_ERR_INVALID_ARG;
  // batch < 0: the most recent forward = the slot with the largest batch index
  int slot = -1;
  for (int i = 0; i < m.D; ++i) {
    if (m.slot_batch[i] < 0) continue;
    if (batch >= 0 ? m.slot_batch[i] == batch : (slot < 0 || m.slot_batch[i] > m.slot_batch[slot])) slot = i;
  }
  *batch_index = slot < 0 ? -1 : m.slot_batch[slot];
  if (slot < 0) return FDG_OK;
  const char* src = m.fifo + ((size_t)slot * m.slot_elems + off) * c->esize;
  return export_tensor(c, src, elems / ch, ch, ch, dst, n);
}

fdg_status fdg_get_saved_tensor(fdg_ctx* c, int module, int unit, int which, float* dst, size_t n, size_t* out_elems,
                                int64_t* batch_index) {
  return fdg_get_saved_tensor_of(c, module, unit, which, -1, dst, n, out_elems, batch_index);
}

fdg_status fdg_capture_bytes(const fdg_ctx* c, int module, size_t* out_bytes) {
  FDG_MODULE_OR_FAIL(c, module);
  if (!out_bytes) return FDG_ERR_INVALID_ARG;
  *out_bytes = c->mods[module - 1].cap_elems * c->esize;
  return FDG_OK;
}

fdg_status fdg_capture_begin(fdg_ctx* c, int module, void* dev_buffer, size_t bytes) {
  FDG_MODULE_OR_FAIL(c, module);
  if (!dev_buffer || (reinterpret_cast<uintptr_t>(dev_buffer) & 15)) return fail(c, FDG_ERR_INVALID_ARG, "capture buffer is null or not 16-byte aligned");
  if (c->use_graphs) return fail(c, FDG_ERR_STATE, "a capture cannot be switched on and off inside recorded graphs");
  Module& m = c->mods[module - 1];
  if (bytes < m.cap_elems * c->esize) return fail(c, FDG_ERR_WORKSPACE_TOO_SMALL, "capture buffer smaller than fdg_capture_bytes");
  cudaError_t e = drain(c);
  if (e != cudaSuccess) return cuda_fail(c, e, "drain");
  m.cap_buf = static_cast<char*>(dev_buffer);
  m.cap_batch = -1;
  return FDG_OK;
}

fdg_status fdg_capture_end(fdg_ctx* c, int module) {
  FDG_MODULE_OR_FAIL(c, module);
  cudaError_t e = drain(c);
  if (e != cudaSuccess) return cuda_fail(c, e, "drain");
  c->mods[module - 1].cap_buf = nullptr;
  return FDG_OK;
}

fdg_status fdg_get_captured(fdg_ctx* c, int module, int unit, int which, float* dst, size_t n, size_t* out_elems,
                            int64_t* batch_index) {
  FDG_MODULE_OR_FAIL(c, module);
  Module& m = c->mods[module - 1];
  const CaptureEntry* ce = nullptr;
  for (const CaptureEntry& x : m.cap_table) if (x.unit == unit && x.which == which) ce = &x;
  if (!ce) return fail(c, FDG_ERR_INVALID_ARG, "this unit's backward produces no such gradient tensor");
  if (out_elems) *out_elems = ce->elems;
  if (!dst) return FDG_OK;
  if (!batch_index) return FDG_ERR_INVALID_ARG;
  if (!m.cap_buf) return fail(c, FDG_ERR_STATE, "no capture is on for this module");
  *batch_index = m.cap_batch;
  if (m.cap_batch < 0) return FDG_OK;
  return export_tensor(c, m.cap_buf + ce->off * c->esize, ce->elems / ce->ch, ce->ch, ce->ch, dst, n);
}

fdg_status fdg_get_schedule_log(const fdg_ctx* c, fdg_sched_entry* dst, size_t cap, size_t* out_n) {
  if (!c) return FDG_ERR_INVALID_ARG;
  if (out_n) *out_n = c->log.size();
  if (dst) for (size_t i = 0; i < std::min(cap, c->log.size()); ++i) dst[i] = c->log[i];
  return FDG_OK;
}

fdg_status fdg_profile_enable(fdg_ctx* c, int on) {
  if (!c) return FDG_ERR_INVALID_ARG;
  if (c->use_graphs && on) return fail(c, FDG_ERR_STATE, "the per-launch profiler cannot time launches replayed from a graph");
  cudaError_t e = drain(c);
  if (e != cudaSuccess) return cuda_fail(c, e, "drain");
  c->profiling = on != 0;
  c->prof_recs.clear();
  return FDG_OK;
}

fdg_status fdg_profile_read(fdg_ctx* c, fdg_kernel_stat* dst, size_t cap, size_t* out_n) {
  if (!c) return FDG_ERR_INVALID_ARG;
  cudaError_t e = drain(c);
  if (e != cudaSuccess) return cuda_fail(c, e, "drain");
  fdg_kernel_stat agg[KC_COUNT];
  for (int i = 0; i < KC_COUNT; ++i) {
    std::memset(&agg[i], 0, sizeof(agg[i]));
    std::snprintf(agg[i].name, sizeof(agg[i].name), "%s", kClassNames[i]);
  }
  for (size_t i = 0; i < c->prof_recs.size(); ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->prof_events[2 * i], c->prof_events[2 * i + 1]) != cudaSuccess) continue;
    fdg_kernel_stat& a = agg[c->prof_recs[i].cls];
    a.launches += 1; a.total_ms += ms; a.bytes += c->prof_recs[i].bytes; a.flops += c->prof_recs[i].flops;
  }
  c->prof_recs.clear();
  if (out_n) *out_n = KC_COUNT;
  if (dst) for (size_t i = 0; i < std::min<size_t>(cap, KC_COUNT); ++i) dst[i] = agg[i];
  return FDG_OK;
}

fdg_status fdg_profile_read_modules(fdg_ctx* c, double* busy_ms, size_t cap, size_t* out_n) {
  if (!c) return FDG_ERR_INVALID_ARG;
  cudaError_t e = drain(c);
  if (e != cudaSuccess) return cuda_fail(c, e, "drain");
  std::vector<double> tot(c->K, 0.0);
  for (size_t i = 0; i < c->mod_event_owner.size(); ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->mod_events[2 * i], c->mod_events[2 * i + 1]) == cudaSuccess) tot[c->mod_event_owner[i]] += ms;
  }
  for (cudaEvent_t ev : c->mod_events) cudaEventDestroy(ev);
  c->mod_events.clear(); c->mod_event_owner.clear();
  if (out_n) *out_n = (size_t)c->K;
  if (busy_ms) for (size_t k = 0; k < std::min<size_t>(cap, (size_t)c->K); ++k) busy_ms[k] = tot[k];
  return FDG_OK;
}

fdg_status fdg_launch_count(const fdg_ctx* c, uint64_t* out_n) {
  if (!c || !out_n) return FDG_ERR_INVALID_ARG;
  *out_n = c->launches;
  return FDG_OK;
}

}  // extern "C"

#include "ops_api.inc"
