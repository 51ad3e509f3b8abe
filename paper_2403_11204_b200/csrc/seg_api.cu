// C ABI of the segment trainer (declared in include/seg.h): handle, workspace layout, and the
// order in which one training step enqueues its kernels.
//
// Device memory layout of a handle
//   params / grads / state1 / state2 : one flat fp32 range each, identical layout
//       [W_0 | b_0 | W_1 | b_1 | ...], every tensor starting on a 256-byte boundary, W_l stored
//       [out][ldw] with ldw = in rounded up to 8 elements (16-byte rows for TMA); padding stays 0.
//   params_op : the same layout in the operand dtype (bf16, or TF32-rounded fp32).
//   act[l], l = 1..L : [max_batch][ld_l] stored outputs (bf16 or fp32; final logits fp32).
//   dzbuf[l]         : dZ of layer l, [max_batch][ld_{l+1}] (one per layer: the weight-gradient
//                      branch reads dZ_l while the main branch already produces dZ_{l-1}).
//   sil              : [M][N_P] fp32 intermediate labels (Eq. 1).
//
// One training step is a dependency graph with one branch per layer.  Main branch: input staging,
// forward products, loss, the dgrad chain, then layer 0's weight gradient and update.  Branch of
// layer l >= 1: the weight-gradient product as soon as dZ_l exists, then the update of W_l and b_l
// (the same launch forms the bias gradient), which also waits for dgrad(l), the last reader of the
// old weights.  The upper layers' HBM-bound updates thereby run beside the tensor-core products of
// the layers below, and only two kernels follow the last dgrad.  After one eager run per batch size
// the step is captured into a CUDA graph and replayed; the caller's x / cls are first copied into
// fixed staging buffers so that the graph never changes.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <stdlib.h>

#include <algorithm>
#include <atomic>
#include <functional>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"

using namespace segk;

namespace {

struct LayerInfo {
  int in, out;
  int64_t ldw;
  int64_t w_off, b_off;  // element offsets into the flat ranges
};

enum Kind { K_FWD = 0, K_DGRAD, K_WGRAD, K_LOSS, K_WGRAD_UPDATE, K_UPDATE, K_COPY, K_FWD_BWD, K_COUNT };   // values are part of the ABI

int64_t round_up(int64_t v, int64_t m) { return (v + m - 1) / m * m; }

// Position of the caller-supplied pointers in the parameter list of the kernel that takes them in: the input
// staging kernel (see elementwise.cu), or the first kernel of a small segment's two-launch step.
struct StageArgs { int count, x, cls, gather, loss; };
constexpr StageArgs kStageInputsArgs = {19, 3, 9, 14, 15};
constexpr StageArgs kSmallStepArgs = {5, 1, 2, 3, 4};

}  // namespace

struct seg_handle {
  int n_layers = 0, n_classes = 0, max_batch = 0, segment_id = 0;
  bool is_final = false, last_relu = false;
  int precision = SEG_FP32, optimizer = SEG_SGD;
  float lr = 0, momentum = 0, beta1 = 0, beta2 = 0, eps = 0;
  uint64_t init_seed = 0;
  cudaStream_t stream = nullptr;
  int device = 0;                  // the device the handle lives on (current when seg_create ran)
  bool use_tc = false;
  bool force_tc = false;           // SEG_GEMM_TCGEN05: a product the tensor-core path cannot take is an error
  uint64_t family_launches[FAM_COUNT] = {0, 0, 0, 0};
  uint64_t fused_updates = 0;      // weight-gradient products that also applied the optimizer update
  int act_dt = DT_F32, act_round = RND_NONE, op_dt = DT_F32, op_round = RND_NONE;
  std::vector<int> widths;
  std::vector<LayerInfo> layers;
  int64_t n_flat = 0;
  float *params = nullptr, *grads = nullptr, *state1 = nullptr, *state2 = nullptr;
  void* params_op = nullptr;
  std::vector<void*> act;          // index 1..L
  std::vector<int64_t> ld_act;     // index 0..L
  std::vector<int> act_dtype;      // index 1..L
  void* x_stage = nullptr;
  int32_t* cls_stage = nullptr;
  std::vector<void*> dzbuf;        // index 0..L-1
  float* loss_slot = nullptr;
  float** loss_dst = nullptr;      // device slot: where the current step's loss goes (filled by the staging launch)
  unsigned long long* step_dev = nullptr;
  float* bc_dev = nullptr;
  // FFMA path: split-K workspaces.  Index 0 serves the main branch (its products run one after another),
  // index l >= 1 the weight gradient of layer l, which runs on its own branch.
  std::vector<float*> simt_scratch;
  std::vector<unsigned int*> simt_counters;
  std::vector<int> simt_slots;
  std::vector<cudaStream_t> lstream;  // lstream[l], l >= 1: the branch of layer l (weight gradient, then update)
  std::vector<cudaEvent_t> ev_dz;     // ev_dz[l]: dZ_l is complete (main branch)
  std::vector<cudaEvent_t> ev_done;   // ev_done[l], l >= 1: layer l's branch is complete
  // A captured step.  The caller's pointers (x, cls, loss_out) enter the graph in one kernel node only,
  // the input staging; its parameters are rewritten before a replay when they differ.
  struct StepGraph {
    int eager_runs = 0;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    uint64_t kernels = 0, kernels_peer = 0;
    uint64_t family[FAM_COUNT] = {0, 0, 0, 0}, family_peer[FAM_COUNT] = {0, 0, 0, 0};
    uint64_t fused = 0;
    seg_handle* peer = nullptr;
    cudaGraphNode_t stage_node = nullptr;
    StageArgs stage_idx{};
    cudaKernelNodeParams stage_params{};
    std::vector<void*> stage_args;
    const void* cur_x = nullptr; const int32_t* cur_cls = nullptr; float* cur_loss = nullptr;   // now in the exec
    const float* cur_gather = nullptr;
  };
  cudaGraphNode_t cap_stage_node = nullptr;   // filled while capturing
  StageArgs cap_stage_idx{};
  bool capturing = false;
  std::map<int, StepGraph> graphs; // by batch size
  std::map<std::pair<uint64_t, int>, StepGraph> recovery_graphs;   // by (right segment's uid, batch size)
  uint64_t uid = 0;                // unique per handle of the process (a reused address is not the same segment)
  bool graphs_enabled = true;
  bool fuse_loss = true;           // take the intermediate-label loss in the last forward product's epilogue where possible
  bool fork_enabled = true;        // run the gradient and update branches on their own streams
  bool small_fused = false;        // small fp32 segment: the whole step runs as two launches (SEG_NO_SMALL_FUSED=1: off)
  SmallStep small{};               // its description, filled by seg_create (batch is set per step)
  bool fuse_update = false;        // SEG_FUSED_UPDATE=1: apply the optimizer inside the weight-gradient product where the
                                   // kernel can (measured slower than the separate update launch, see gemm_tc.cu)
  float* sil = nullptr;
  bool have_labels = false;
  float* loss_partials = nullptr;
  unsigned int* loss_counter = nullptr;
  int* dev_status = nullptr;
  void* host_x = nullptr;          // device staging of seg_train_step_host
  int32_t* host_cls = nullptr;
  float* host_loss = nullptr;      // page-locked host float the loss kernel writes (seg_train_step_host)
  float* host_loss_dev = nullptr;  // its device-side address
  // seg_train_step_host_async: copy stream, two device buffers for the batch in flight and the next one
  cudaStream_t copy_stream = nullptr;
  void* async_x[2] = {nullptr, nullptr};
  int32_t* async_cls[2] = {nullptr, nullptr};
  cudaEvent_t ev_copied[2] = {nullptr, nullptr}, ev_consumed[2] = {nullptr, nullptr};
  bool async_used[2] = {false, false};
  int async_next = 0;
  int last_batch = 0;
  uint64_t step = 0;
  uint64_t mem_current = 0, mem_peak = 0, launches = 0;
  std::vector<void*> allocations;
  cudaEvent_t ev_start = nullptr, ev_stop = nullptr;
  cudaEvent_t ev_handoff = nullptr;   // seg_handoff_copy: the copy out of this handle's device is complete
  bool profile = false;
  std::vector<cudaEvent_t> ev_pool;
  size_t ev_used = 0;
  std::vector<int> ev_kind;        // kind of each recorded pair
  std::string last_error;
};

namespace {

// Makes the handle's device current for the duration of one call and restores the caller's.
struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  explicit DeviceGuard(const seg_handle* h) {
    if (!h) return;
    if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); return; }
    if (prev != h->device && cudaSetDevice(h->device) == cudaSuccess) switched = true;
  }
  ~DeviceGuard() { if (switched) cudaSetDevice(prev); }
};

seg_status fail_cuda(seg_handle* h, cudaError_t e, const char* what) {
  if (h) h->last_error = std::string(what) + ": " + cudaGetErrorString(e);
  return e == cudaErrorMemoryAllocation ? SEG_ERR_ALLOC : SEG_ERR_CUDA;
}

#define SEG_TRY(h, expr, what)                                   \
  do {                                                           \
    cudaError_t e__ = (expr);                                    \
    if (e__ != cudaSuccess) return fail_cuda((h), e__, (what));  \
  } while (0)

template <typename T>
seg_status dev_alloc(seg_handle* h, T** out, size_t count, bool zero) {
  const size_t bytes = round_up((int64_t)(count * sizeof(T)), 256);
  void* p = nullptr;
  if (bytes == 0) { *out = nullptr; return SEG_OK; }
  cudaError_t e = cudaMalloc(&p, bytes);
  if (e != cudaSuccess) { cudaGetLastError(); return fail_cuda(h, e, "cudaMalloc"); }
  h->allocations.push_back(p);
  h->mem_current += bytes;
  if (h->mem_current > h->mem_peak) h->mem_peak = h->mem_current;
  if (zero) SEG_TRY(h, cudaMemsetAsync(p, 0, bytes, h->stream), "cudaMemsetAsync");
  *out = reinterpret_cast<T*>(p);
  return SEG_OK;
}

// Brackets one launch with events while profiling is on.
struct Launch {
  seg_handle* h;
  bool on;
  cudaStream_t st;
  Launch(seg_handle* hh, int kind, cudaStream_t stream = nullptr)
      : h(hh), on(hh->profile), st(stream ? stream : hh->stream) {
    ++h->launches;
    if (!on) return;
    if (h->ev_used + 2 > h->ev_pool.size()) {
      for (int i = 0; i < 2; ++i) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess) { on = false; return; }
        h->ev_pool.push_back(e);
      }
    }
    cudaEventRecord(h->ev_pool[h->ev_used], st);
    h->ev_kind.push_back(kind);
  }
  ~Launch() {
    if (!on) return;
    cudaEventRecord(h->ev_pool[h->ev_used + 1], st);
    h->ev_used += 2;
  }
};

seg_status run_gemm(seg_handle* h, const GemmDesc& g_in, int kind, cudaStream_t stream, bool* used_tc = nullptr,
                    int workspace = 0) {
  Launch l(h, kind, stream);
  if (used_tc) *used_tc = false;
  GemmDesc g = g_in;
  if (workspace < (int)h->simt_scratch.size() && h->simt_scratch[workspace]) {
    g.simt_scratch = h->simt_scratch[workspace]; g.simt_counters = h->simt_counters[workspace];
    g.simt_slots = h->simt_slots[workspace];
  }
  if (h->use_tc) {
    int family = FAM_TC_SINGLE;
    cudaError_t e = launch_gemm_tc(g, h->dev_status, stream, &family);
    if (e == cudaSuccess) { if (used_tc) *used_tc = true; ++h->family_launches[family]; return SEG_OK; }
    if (e != cudaErrorNotSupported) return fail_cuda(h, e, "tensor-core product launch");
    cudaGetLastError();
    if (h->force_tc) {
      h->last_error = "the tensor-core path cannot take this product (operand alignment or strides) and the handle "
                      "was created with SEG_GEMM_TCGEN05";
      return SEG_ERR_UNSUPPORTED;
    }
  }
  SEG_TRY(h, launch_gemm_simt(g, stream), "FFMA product launch");
  ++h->family_launches[FAM_SIMT];
  return SEG_OK;
}

size_t elem_size(int dt) { return dt == DT_BF16 ? 2 : 4; }

void* weights_op(seg_handle* h, int l) {
  char* base = reinterpret_cast<char*>(h->params_op ? h->params_op : (void*)h->params);
  return base + h->layers[l].w_off * elem_size(h->params_op ? h->op_dt : DT_F32);
}

// Returns the pointer / pitch the first product reads x from, staging it when the caller's
// buffer cannot be used directly (TF32 rounding, or rows that are not 16-byte multiples).
seg_status prepare_input(seg_handle* h, const void* x, int batch, const void** x_use, int64_t* ld) {
  const int w0 = h->widths[0];
  const bool aligned = ((reinterpret_cast<uintptr_t>(x) & 15u) == 0) &&
                       ((w0 * elem_size(h->act_dt)) % 16 == 0);
  if (h->precision != SEG_TF32 && (aligned || !h->use_tc)) {
    *x_use = x; *ld = w0;
    return SEG_OK;
  }
  Launch l(h, K_COPY);
  SEG_TRY(h, launch_copy2d(h->x_stage, h->act_dt, h->ld_act[0], x, h->act_dt, w0, batch, w0,
                           h->act_round, h->stream), "input staging");
  *x_use = h->x_stage; *ld = h->ld_act[0];
  return SEG_OK;
}

// Description of a non-final segment's loss for fusion into its last forward product.
LossFuse loss_fuse_desc(seg_handle* h, int batch, const int32_t* cls, float* const* loss_dst) {
  const int L = h->n_layers;
  LossFuse f{};
  f.enabled = 1;
  f.cls = cls; f.sil = h->sil;
  f.dz = h->dzbuf[L - 1]; f.ld_dz = h->ld_act[L]; f.dz_dt = h->act_dt; f.dz_round = h->act_round;
  f.relu_mask = h->last_relu ? 1 : 0;
  const double count = (double)batch * h->widths[L];
  f.gscale = 2.0f / (float)((int64_t)batch * h->widths[L]);
  f.loss_scale = (float)(1.0 / count);
  f.partials = h->loss_partials; f.counter = h->loss_counter; f.loss_dst = loss_dst;
  return f;
}

// The segment's loss as a launch of its own (the final segment's softmax cross-entropy always; the
// intermediate-label loss when the last forward product could not take it).
seg_status launch_loss(seg_handle* h, int batch, const int32_t* cls, float* const* loss_dst) {
  const int L = h->n_layers;
  Launch l(h, K_LOSS, h->stream);
  void* dz_L = h->dzbuf[L - 1];
  if (h->is_final) {
    SEG_TRY(h, launch_softmax_ce_loss((const float*)h->act[L], h->ld_act[L], cls, h->n_classes, batch,
                                      h->last_relu ? 1 : 0, dz_L, h->act_dt, h->act_round, h->ld_act[L],
                                      h->loss_partials, h->loss_counter, loss_dst, h->stream), "softmax-CE loss");
  } else {
    SEG_TRY(h, launch_mse_loss(h->act[L], h->act_dtype[L], h->ld_act[L], cls, h->sil, h->n_classes, h->widths[L], batch,
                               h->last_relu ? 1 : 0, dz_L, h->act_dt, h->act_round, h->ld_act[L],
                               h->loss_partials, h->loss_counter, loss_dst, h->stream), "MSE loss");
  }
  return SEG_OK;
}

// Forward products of all layers, reading layer 0's input from (a_prev, ld_prev).  With loss_cls not
// null the segment's loss follows: inside the last product's epilogue where the tensor-core path can
// take it, as a separate launch otherwise.
seg_status forward_layers(seg_handle* h, const void* a_prev, int64_t ld_prev, int batch,
                          const int32_t* loss_cls = nullptr, float* const* loss_dst = nullptr) {
  for (int l = 0; l < h->n_layers; ++l) {
    const LayerInfo& L = h->layers[l];
    const bool last = (l == h->n_layers - 1);
    GemmDesc g{};
    g.A = a_prev; g.a_sm = ld_prev; g.a_sk = 1; g.a_dt = h->act_dt;
    g.B = weights_op(h, l); g.b_sk = 1; g.b_sn = L.ldw; g.b_dt = h->op_dt;
    g.C = h->act[l + 1]; g.ldc = h->ld_act[l + 1]; g.c_dt = h->act_dtype[l + 1];
    g.M = batch; g.N = L.out; g.K = L.in;
    g.c_round = (last && h->is_final) ? RND_NONE : h->act_round;
    g.epi = EPI_BIAS_ACT; g.relu = (!last || h->last_relu) ? 1 : 0;
    g.bias = h->params + L.b_off;
    const bool want_loss = last && loss_cls != nullptr;
    if (want_loss && !h->is_final && h->use_tc && h->fuse_loss &&
        gemm_tc_can_fuse_loss(g.M, g.N, g.K, h->precision == SEG_TF32))
      g.loss = loss_fuse_desc(h, batch, loss_cls, loss_dst);
    bool used_tc = false;
    seg_status st = run_gemm(h, g, K_FWD, h->stream, &used_tc);
    if (st != SEG_OK) return st;
    if (want_loss && !(used_tc && g.loss.enabled) && (st = launch_loss(h, batch, loss_cls, loss_dst)) != SEG_OK) return st;
    a_prev = h->act[l + 1]; ld_prev = h->ld_act[l + 1];
  }
  h->last_batch = batch;
  return SEG_OK;
}

seg_status forward_impl(seg_handle* h, const void* x, int batch) {
  const void* a_prev; int64_t ld_prev;
  seg_status st = prepare_input(h, x, batch, &a_prev, &ld_prev);
  if (st != SEG_OK) return st;
  return forward_layers(h, a_prev, ld_prev, batch);
}

seg_status copy_out(seg_handle* h, void* y, int batch) {
  const int L = h->n_layers;
  Launch l(h, K_COPY);
  SEG_TRY(h, launch_copy2d(y, h->act_dtype[L], h->widths[L], h->act[L], h->act_dtype[L],
                           h->ld_act[L], batch, h->widths[L], RND_NONE, h->stream), "output copy");
  return SEG_OK;
}

seg_status refresh_operand_copy(seg_handle* h, int64_t off, int64_t n) {
  if (!h->params_op || n == 0) return SEG_OK;
  Launch l(h, K_COPY);
  char* dst = reinterpret_cast<char*>(h->params_op) + off * elem_size(h->op_dt);
  SEG_TRY(h, launch_copy2d(dst, h->op_dt, n, h->params + off, DT_F32, n, 1, n, h->op_round,
                           h->stream), "operand copy refresh");
  return SEG_OK;
}

bool valid_layer(const seg_handle* h, int layer) { return layer >= 0 && layer < h->n_layers; }

}  // namespace

extern "C" {

const char* seg_status_string(int32_t s) {
  switch (s) {
    case SEG_OK: return "ok";
    case SEG_ERR_INVALID_ARG: return "invalid argument";
    case SEG_ERR_SHAPE: return "shape out of range";
    case SEG_ERR_UNSUPPORTED: return "unsupported configuration";
    case SEG_ERR_ALLOC: return "device allocation failed";
    case SEG_ERR_CUDA: return "CUDA call failed";
    case SEG_ERR_STATE: return "call not valid in this state";
    case SEG_ERR_DEVICE_TIMEOUT: return "a kernel gave up a bounded wait";
    case SEG_ERR_NO_DEVICE: return "no usable CUDA device";
    case SEG_ERR_CLASS_RANGE: return "class index outside [0, n_classes)";
    default: return "unknown status";
  }
}

const char* seg_build_info(void) { return "segment trainer for sm_100a (tcgen05/TMEM/TMA products, FFMA fp32 path)"; }

const char* seg_last_error(const seg_handle* h) { return h ? h->last_error.c_str() : ""; }

seg_status seg_create(const seg_config* cfg, seg_handle** out) {
  if (!out) return SEG_ERR_INVALID_ARG;
  *out = nullptr;
  if (!cfg || !cfg->widths) return SEG_ERR_INVALID_ARG;
  if (cfg->n_layers < 1 || cfg->n_layers > 16) return SEG_ERR_SHAPE;
  if (cfg->n_classes < 1 || cfg->max_batch < 1) return SEG_ERR_SHAPE;
  for (int i = 0; i <= cfg->n_layers; ++i)
    if (cfg->widths[i] < 1 || cfg->widths[i] > (1 << 20)) return SEG_ERR_SHAPE;
  if (cfg->precision < SEG_FP32 || cfg->precision > SEG_BF16) return SEG_ERR_INVALID_ARG;
  if (cfg->optimizer < SEG_SGD || cfg->optimizer > SEG_ADAM) return SEG_ERR_INVALID_ARG;
  if (cfg->gemm_backend < SEG_GEMM_AUTO || cfg->gemm_backend > SEG_GEMM_TCGEN05) return SEG_ERR_INVALID_ARG;
  if (cfg->gemm_backend == SEG_GEMM_TCGEN05 && cfg->precision == SEG_FP32) return SEG_ERR_UNSUPPORTED;
  if (cfg->is_final && cfg->widths[cfg->n_layers] != cfg->n_classes) return SEG_ERR_SHAPE;
  if (!(cfg->lr >= 0.f)) return SEG_ERR_INVALID_ARG;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SEG_ERR_NO_DEVICE; }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { cudaGetLastError(); return SEG_ERR_NO_DEVICE; }
  if (prop.major != 10) return SEG_ERR_NO_DEVICE;

  seg_handle* h = new (std::nothrow) seg_handle();
  if (!h) return SEG_ERR_ALLOC;
  static std::atomic<uint64_t> next_uid{0};
  h->uid = ++next_uid;
  h->device = dev;
  h->force_tc = cfg->gemm_backend == SEG_GEMM_TCGEN05;
  h->n_layers = cfg->n_layers; h->n_classes = cfg->n_classes; h->max_batch = cfg->max_batch;
  h->segment_id = cfg->segment_id; h->is_final = cfg->is_final != 0;
  h->last_relu = cfg->last_relu < 0 ? !h->is_final : (cfg->last_relu != 0);
  h->precision = cfg->precision; h->optimizer = cfg->optimizer;
  h->lr = cfg->lr; h->momentum = cfg->momentum; h->beta1 = cfg->beta1; h->beta2 = cfg->beta2;
  h->eps = cfg->eps; h->init_seed = cfg->init_seed;
  h->stream = reinterpret_cast<cudaStream_t>(cfg->stream);
  h->widths.assign(cfg->widths, cfg->widths + cfg->n_layers + 1);
  if (h->precision == SEG_BF16) { h->act_dt = DT_BF16; h->act_round = RND_BF16; h->op_dt = DT_BF16; h->op_round = RND_BF16; }
  if (h->precision == SEG_TF32) { h->act_round = RND_TF32; h->op_round = RND_TF32; }
  h->use_tc = (h->precision != SEG_FP32) && (cfg->gemm_backend != SEG_GEMM_SIMT);
  if (h->use_tc && !gemm_tc_init()) {
    if (cfg->gemm_backend == SEG_GEMM_TCGEN05) { delete h; return SEG_ERR_UNSUPPORTED; }
    h->use_tc = false;
  }

  seg_status st = SEG_OK;
  auto bail = [&](seg_status s) { seg_destroy(h); return s; };

  int64_t off = 0;
  for (int l = 0; l < h->n_layers; ++l) {
    LayerInfo L;
    L.in = h->widths[l]; L.out = h->widths[l + 1];
    L.ldw = round_up(L.in, 8);
    L.w_off = off; off = round_up(off + (int64_t)L.out * L.ldw, 64);
    L.b_off = off; off = round_up(off + L.out, 64);
    h->layers.push_back(L);
  }
  h->n_flat = off;
  if ((st = dev_alloc(h, &h->params, h->n_flat, true)) != SEG_OK) return bail(st);
  if ((st = dev_alloc(h, &h->grads, h->n_flat, true)) != SEG_OK) return bail(st);
  if (h->optimizer != SEG_SGD && (st = dev_alloc(h, &h->state1, h->n_flat, true)) != SEG_OK) return bail(st);
  if (h->optimizer == SEG_ADAM && (st = dev_alloc(h, &h->state2, h->n_flat, true)) != SEG_OK) return bail(st);
  if (h->precision != SEG_FP32) {
    char* p = nullptr;
    if ((st = dev_alloc(h, &p, h->n_flat * elem_size(h->op_dt), true)) != SEG_OK) return bail(st);
    h->params_op = p;
  }
  h->act.assign(h->n_layers + 1, nullptr);
  h->ld_act.assign(h->n_layers + 1, 0);
  h->act_dtype.assign(h->n_layers + 1, h->act_dt);
  for (int l = 0; l <= h->n_layers; ++l) {
    h->ld_act[l] = round_up(h->widths[l], 8);
  }
  if (h->is_final) h->act_dtype[h->n_layers] = DT_F32;
  for (int l = 1; l <= h->n_layers; ++l) {
    char* p = nullptr;
    const size_t bytes = (size_t)h->max_batch * h->ld_act[l] * elem_size(h->act_dtype[l]);
    if ((st = dev_alloc(h, &p, bytes, true)) != SEG_OK) return bail(st);
    h->act[l] = p;
  }
  {
    char* p = nullptr;
    if ((st = dev_alloc(h, &p, (size_t)h->max_batch * h->ld_act[0] * elem_size(h->act_dt), true)) != SEG_OK) return bail(st);
    h->x_stage = p;
  }
  h->dzbuf.assign(h->n_layers, nullptr);
  for (int l = 0; l < h->n_layers; ++l) {
    char* p = nullptr;
    if ((st = dev_alloc(h, &p, (size_t)h->max_batch * h->ld_act[l + 1] * elem_size(h->act_dt), true)) != SEG_OK) return bail(st);
    h->dzbuf[l] = p;
  }
  if ((st = dev_alloc(h, &h->cls_stage, h->max_batch, true)) != SEG_OK) return bail(st);
  if ((st = dev_alloc(h, &h->loss_slot, 1, true)) != SEG_OK) return bail(st);
  if ((st = dev_alloc(h, &h->loss_dst, 1, true)) != SEG_OK) return bail(st);
  if ((st = dev_alloc(h, &h->step_dev, 1, true)) != SEG_OK) return bail(st);
  if ((st = dev_alloc(h, &h->bc_dev, 2, true)) != SEG_OK) return bail(st);
  h->lstream.assign(h->n_layers, nullptr);
  h->ev_dz.assign(h->n_layers, nullptr);
  h->ev_done.assign(h->n_layers, nullptr);
  for (int l = 0; l < h->n_layers; ++l) {
    if (l > 0 && cudaStreamCreateWithFlags(&h->lstream[l], cudaStreamNonBlocking) != cudaSuccess) return bail(SEG_ERR_CUDA);
    if (cudaEventCreateWithFlags(&h->ev_dz[l], cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_done[l], cudaEventDisableTiming) != cudaSuccess) return bail(SEG_ERR_CUDA);
  }
  {
    const char* env = getenv("SEG_NO_GRAPH");
    if (env && env[0] == '1') h->graphs_enabled = false;
    static std::once_flag pdl_once;      // process-wide switch: written once, before any launch of any handle
    std::call_once(pdl_once, [] {
      const char* e = getenv("SEG_NO_PDL");
      if (e && e[0] == '1') g_use_pdl = false;
    });
    env = getenv("SEG_NO_FORK");
    if (env && env[0] == '1') h->fork_enabled = false;
    env = getenv("SEG_NO_FUSED_LOSS");
    if (env && env[0] == '1') h->fuse_loss = false;
    env = getenv("SEG_FUSED_UPDATE");
    if (env && env[0] == '1') h->fuse_update = true;
  }
  if (!h->use_tc) {
    // split-K workspaces of the FFMA path, sized for the products each one serves at max_batch
    h->simt_scratch.assign(h->n_layers, nullptr);
    h->simt_counters.assign(h->n_layers, nullptr);
    h->simt_slots.assign(h->n_layers, 0);
    const int B = h->max_batch;
    for (int l = 0; l < h->n_layers; ++l) {
      const int in = h->widths[l], out = h->widths[l + 1];
      const int wg = gemm_simt_slots(out, in, B);
      if (l > 0) h->simt_slots[l] = wg;
      else h->simt_slots[0] = std::max(h->simt_slots[0], wg);
      h->simt_slots[0] = std::max(h->simt_slots[0], gemm_simt_slots(B, out, in));            // forward
      if (l > 0) h->simt_slots[0] = std::max(h->simt_slots[0], gemm_simt_slots(B, in, out)); // dgrad
    }
    for (int l = 0; l < h->n_layers; ++l) {
      if (h->simt_slots[l] == 0) continue;
      if ((st = dev_alloc(h, &h->simt_scratch[l], (size_t)h->simt_slots[l] * kSimtTileFloats, false)) != SEG_OK) return bail(st);
      if ((st = dev_alloc(h, &h->simt_counters[l], h->simt_slots[l], true)) != SEG_OK) return bail(st);
    }
  }
  if (!h->is_final &&
      (st = dev_alloc(h, &h->sil, (size_t)h->n_classes * h->widths[h->n_layers], true)) != SEG_OK) return bail(st);
  if ((st = dev_alloc(h, &h->loss_partials, loss_max_partials(), true)) != SEG_OK) return bail(st);
  if ((st = dev_alloc(h, &h->loss_counter, 1, true)) != SEG_OK) return bail(st);
  if ((st = dev_alloc(h, &h->dev_status, 1, true)) != SEG_OK) return bail(st);
  {
    const char* env = getenv("SEG_NO_SMALL_FUSED");
    h->small_fused = h->precision == SEG_FP32 && !(env && env[0] == '1') &&
                     small_step_supported(h->n_layers, h->widths.data());
  }
  if (h->small_fused) {
    SmallStep& p = h->small;
    p.n_layers = h->n_layers; p.n_classes = h->n_classes; p.is_final = h->is_final ? 1 : 0;
    p.last_relu = h->last_relu ? 1 : 0; p.optimizer = h->optimizer;
    for (int l = 0; l <= h->n_layers; ++l) {
      p.widths[l] = h->widths[l]; p.ld_act[l] = h->ld_act[l];
      p.act[l] = reinterpret_cast<float*>(l == 0 ? h->x_stage : h->act[l]);
    }
    for (int l = 0; l < h->n_layers; ++l) {
      p.ldw[l] = h->layers[l].ldw; p.w_off[l] = h->layers[l].w_off; p.b_off[l] = h->layers[l].b_off;
      p.dz[l] = reinterpret_cast<float*>(h->dzbuf[l]);
    }
    p.params = h->params; p.grads = h->grads; p.s1 = h->state1; p.s2 = h->state2;
    p.sil = h->sil; p.cls_stage = h->cls_stage;
    p.loss_partials = h->loss_partials; p.loss_counter = h->loss_counter; p.loss_dst = h->loss_dst;
    p.t = h->step_dev; p.bc = h->bc_dev; p.dev_status = h->dev_status;
    p.lr = h->lr; p.momentum = h->momentum; p.beta1 = h->beta1; p.beta2 = h->beta2; p.eps = h->eps;
    p.wg_slots = small_step_wgrad_slots(h->n_layers, h->widths.data());
    if ((st = dev_alloc(h, &p.wg_scratch, (size_t)p.wg_slots * kSimtTileFloats, false)) != SEG_OK) return bail(st);
    if ((st = dev_alloc(h, &p.wg_counters, p.wg_slots, true)) != SEG_OK) return bail(st);
  }
  if (cudaEventCreate(&h->ev_start) != cudaSuccess || cudaEventCreate(&h->ev_stop) != cudaSuccess)
    return bail(SEG_ERR_CUDA);

  for (int l = 0; l < h->n_layers; ++l) {
    const LayerInfo& L = h->layers[l];
    const float bound = 1.0f / sqrtf((float)L.in);
    ++h->launches;
    if (launch_init_uniform(h->params + L.w_off, L.out, L.in, L.ldw, h->init_seed, h->segment_id, l, 1,
                            bound, h->stream) != cudaSuccess) return bail(SEG_ERR_CUDA);
    ++h->launches;
    if (launch_init_uniform(h->params + L.b_off, 1, L.out, L.out, h->init_seed, h->segment_id, l, 2,
                            bound, h->stream) != cudaSuccess) return bail(SEG_ERR_CUDA);
  }
  if ((st = refresh_operand_copy(h, 0, h->n_flat)) != SEG_OK) return bail(st);
  *out = h;
  return SEG_OK;
}

seg_status seg_destroy(seg_handle* h) {
  if (!h) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (h->ev_handoff) cudaEventDestroy(h->ev_handoff);
  if (h->copy_stream) cudaStreamSynchronize(h->copy_stream);
  cudaStreamSynchronize(h->stream);
  for (cudaStream_t ls : h->lstream) if (ls) cudaStreamSynchronize(ls);
  for (auto& kv : h->graphs) {
    if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
    if (kv.second.graph) cudaGraphDestroy(kv.second.graph);
  }
  for (auto& kv : h->recovery_graphs) {
    if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
    if (kv.second.graph) cudaGraphDestroy(kv.second.graph);
  }
  for (cudaEvent_t e : h->ev_dz) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : h->ev_done) if (e) cudaEventDestroy(e);
  for (cudaStream_t ls : h->lstream) if (ls) cudaStreamDestroy(ls);
  for (void* p : h->allocations) cudaFree(p);
  if (h->host_loss) cudaFreeHost(h->host_loss);
  for (int i = 0; i < 2; ++i) {
    if (h->ev_copied[i]) cudaEventDestroy(h->ev_copied[i]);
    if (h->ev_consumed[i]) cudaEventDestroy(h->ev_consumed[i]);
  }
  if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
  for (cudaEvent_t e : h->ev_pool) cudaEventDestroy(e);
  if (h->ev_start) cudaEventDestroy(h->ev_start);
  if (h->ev_stop) cudaEventDestroy(h->ev_stop);
  cudaGetLastError();
  delete h;
  return SEG_OK;
}

seg_status seg_gen_labels(seg_handle* h, uint64_t seed, int32_t dist, float kappa) {
  if (!h) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (h->is_final) return SEG_ERR_STATE;
  if (dist != SEG_LABEL_UNIFORM_KAPPA && dist != SEG_LABEL_NORMAL) return SEG_ERR_INVALID_ARG;
  Launch l(h, K_COPY);
  SEG_TRY(h, launch_gen_labels(h->sil, h->n_classes, h->widths[h->n_layers], seed, h->segment_id, dist,
                               kappa, h->stream), "label generation");
  h->have_labels = true;
  return SEG_OK;
}

seg_status seg_forward(seg_handle* h, const void* x, int32_t batch, void* y) {
  if (!h || !x || !y) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (batch < 1 || batch > h->max_batch) return SEG_ERR_SHAPE;
  seg_status st = forward_impl(h, x, batch);
  if (st != SEG_OK) return st;
  return copy_out(h, y, batch);
}

// Enqueues one whole step (forward, loss, backward, update) that reads the staged inputs.
// forked = false puts all three branches on the main stream (used while profiling).
static cudaGraphNode_t last_captured_node(seg_handle* h) {
  cudaStreamCaptureStatus status;
  unsigned long long id = 0;
  cudaGraph_t graph = nullptr;
  const cudaGraphNode_t* deps = nullptr;
  size_t n = 0;
  if (cudaStreamGetCaptureInfo(h->stream, &status, &id, &graph, &deps, &n) != cudaSuccess || n != 1) {
    cudaGetLastError();
    return nullptr;
  }
  return deps[0];
}

static seg_status enqueue_backward(seg_handle* h, int batch, bool forked);

static seg_status enqueue_step(seg_handle* h, int batch, bool forked, const void* x, const int32_t* cls,
                               float* loss_out, const float* gather) {
  cudaStream_t mainst = h->stream;
  seg_status st;
  float* loss_to = loss_out ? loss_out : h->loss_slot;
  if (h->small_fused && small_step_batch_ok(batch)) {
    // small fp32 segment: staging, forward, loss and the dgrad chain in one launch, every weight and bias
    // gradient with its update in a second
    SmallStep p = h->small;
    p.batch = batch;
    {
      Launch lf(h, K_FWD_BWD);
      SEG_TRY(h, launch_small_fwd_bwd(p, reinterpret_cast<const float*>(x), cls, gather, loss_to, mainst),
              "small-segment forward/backward launch");
    }
    if (h->capturing) { h->cap_stage_node = last_captured_node(h); h->cap_stage_idx = kSmallStepArgs; }
    {
      Launch lw(h, K_WGRAD_UPDATE);
      SEG_TRY(h, launch_small_wgrad_update(p, mainst), "small-segment weight-gradient/update launch");
    }
    h->family_launches[FAM_SIMT] += 2;
    ++h->fused_updates;
    h->last_batch = batch;
    return SEG_OK;
  }
  {
    // fixed staging buffers: rounds x in TF32 mode, pads the pitch, keeps every later pointer constant;
    // the same launch advances the device-side step counter and Adam's bias corrections and records
    // where this step's loss goes
    Launch lc(h, K_COPY);
    SEG_TRY(h, launch_stage_inputs(h->x_stage, h->act_dt, h->ld_act[0], x, h->widths[0], batch, h->widths[0],
                                   h->act_round, h->cls_stage, cls, h->step_dev, h->bc_dev, h->beta1, h->beta2,
                                   gather, loss_to, h->loss_dst, h->n_classes, h->dev_status, mainst), "input staging");
  }
  if (h->capturing) { h->cap_stage_node = last_captured_node(h); h->cap_stage_idx = kStageInputsArgs; }
  if ((st = forward_layers(h, h->x_stage, h->ld_act[0], batch, h->cls_stage, h->loss_dst)) != SEG_OK) return st;
  return enqueue_backward(h, batch, forked);
}

// Backward pass and update of every layer, starting from dZ of the last layer in dzbuf[L-1].
// The main branch carries the dgrad chain and then layer 0's weight gradient and update, all linked
// by programmatic dependent launches.  Every layer l >= 1 has a branch of its own: its weight
// gradient starts as soon as dZ_l exists, its update (which also forms the bias gradient) follows
// once dgrad(l), the last reader of the old W_l, is done.  The branches of the upper layers thereby
// finish beside the dgrad chain, and what is left after the last dgrad is two kernels.
static seg_status enqueue_backward(seg_handle* h, int batch, bool forked) {
  const int L = h->n_layers;
  cudaStream_t mainst = h->stream;
  seg_status st;
  if (forked && L > 1) SEG_TRY(h, cudaEventRecord(h->ev_dz[L - 1], mainst), "event record");
  for (int l = L - 1; l >= 0; --l) {
    const LayerInfo& Ly = h->layers[l];
    const int64_t ld_dz = h->ld_act[l + 1];
    const void* dz_l = h->dzbuf[l];
    const void* a_prev = (l == 0) ? h->x_stage : h->act[l];
    const int64_t ld_prev = h->ld_act[l];
    const bool branch = forked && l > 0;
    cudaStream_t ls = branch ? h->lstream[l] : mainst;
    // main branch first: dgrad of layer l
    if (l > 0) {
      GemmDesc d{};
      d.A = dz_l; d.a_sm = ld_dz; d.a_sk = 1; d.a_dt = h->act_dt;
      d.B = weights_op(h, l); d.b_sk = Ly.ldw; d.b_sn = 1; d.b_dt = h->op_dt;
      d.C = h->dzbuf[l - 1]; d.ldc = h->ld_act[l]; d.c_dt = h->act_dt; d.c_round = h->act_round;
      d.M = batch; d.N = Ly.in; d.K = Ly.out; d.epi = EPI_MASK;
      d.mask = h->act[l]; d.ldmask = h->ld_act[l];
      if ((st = run_gemm(h, d, K_DGRAD, mainst)) != SEG_OK) return st;
      if (forked) SEG_TRY(h, cudaEventRecord(h->ev_dz[l - 1], mainst), "event record");
    }
    // weight gradient of layer l (needs dZ_l)
    if (branch) SEG_TRY(h, cudaStreamWaitEvent(ls, h->ev_dz[l], 0), "stream wait");
    GemmDesc w{};
    w.A = dz_l; w.a_sm = 1; w.a_sk = ld_dz; w.a_dt = h->act_dt;
    w.B = a_prev; w.b_sk = ld_prev; w.b_sn = 1; w.b_dt = h->act_dt;
    w.C = h->grads + Ly.w_off; w.ldc = Ly.ldw; w.c_dt = DT_F32; w.c_round = RND_NONE;
    w.M = Ly.out; w.N = Ly.in; w.K = batch; w.epi = EPI_PLAIN;
    w.off_critical_path = l > 0;  // the upper layers' weight gradients run beside the dgrad chain and each other
    const int64_t lo = Ly.w_off;
    // Opt-in (SEG_FUSED_UPDATE=1; measured slower): where the persistent tensor-core kernels run the product, they also
    // apply the optimizer to W_l (extra warps stream over every stored tile); the launch below then only has the bias
    // left.  The update overwrites W_l's operand copy, which dgrad(l) reads: the fused product waits for dgrad(l), the
    // separate update does the same one launch later.
    const bool fused = h->use_tc && h->fuse_update && h->params_op != nullptr && gemm_tc_can_fuse_update(w);
    if (fused) {
      if (branch) SEG_TRY(h, cudaStreamWaitEvent(ls, h->ev_dz[l - 1], 0), "stream wait");
      FusedUpdate& f = w.upd;
      f.enabled = 1;
      f.p = h->params + lo;
      f.s1 = h->state1 ? h->state1 + lo : nullptr; f.s2 = h->state2 ? h->state2 + lo : nullptr;
      f.p_op = reinterpret_cast<char*>(h->params_op) + lo * elem_size(h->op_dt);
      f.op_dt = h->op_dt; f.op_round = h->op_round; f.optimizer = h->optimizer;
      f.lr = h->lr; f.momentum = h->momentum; f.beta1 = h->beta1; f.beta2 = h->beta2; f.eps = h->eps;
      f.bc = h->bc_dev;
    }
    bool w_on_tc = false;
    if ((st = run_gemm(h, w, fused ? K_WGRAD_UPDATE : K_WGRAD, ls, &w_on_tc, l)) != SEG_OK) return st;
    if (fused && !w_on_tc) { h->last_error = "fused update product did not run on the tensor-core path"; return SEG_ERR_STATE; }
    if (fused) ++h->fused_updates;
    // update of W_l and b_l (adjacent in the flat range) once dgrad(l) no longer reads the old W_l
    if (branch && !fused) SEG_TRY(h, cudaStreamWaitEvent(ls, h->ev_dz[l - 1], 0), "stream wait");
    UpdateArgs u{};
    u.p = h->params + lo; u.g = h->grads + lo;
    u.s1 = h->state1 ? h->state1 + lo : nullptr; u.s2 = h->state2 ? h->state2 + lo : nullptr;
    u.p_op = h->params_op ? (void*)(reinterpret_cast<char*>(h->params_op) + lo * elem_size(h->op_dt)) : nullptr;
    u.op_dt = h->op_dt; u.op_round = h->op_round;
    u.n = fused ? 0 : Ly.b_off - lo; u.optimizer = h->optimizer;
    u.dz = dz_l; u.dz_dt = h->act_dt; u.ld_dz = ld_dz; u.batch = batch; u.n_bias = Ly.out;
    u.bias_off = Ly.b_off - lo; u.g_bias = h->grads + Ly.b_off;
    u.lr = h->lr; u.momentum = h->momentum; u.beta1 = h->beta1; u.beta2 = h->beta2; u.eps = h->eps;
    u.bc = h->bc_dev;
    {
      Launch lu(h, K_UPDATE, ls);
      SEG_TRY(h, launch_update(u, ls), "optimizer update");
    }
    if (branch) SEG_TRY(h, cudaEventRecord(h->ev_done[l], ls), "event record");
  }
  if (forked)
    for (int l = 1; l < L; ++l) SEG_TRY(h, cudaStreamWaitEvent(mainst, h->ev_done[l], 0), "stream wait");
  return SEG_OK;
}

static bool adopt_captured_graph(seg_handle* h, seg_handle::StepGraph& g, cudaGraph_t graph) {
  if (!h->cap_stage_node) return false;
  g.stage_node = h->cap_stage_node;
  g.stage_idx = h->cap_stage_idx;
  if (cudaGraphKernelNodeGetParams(g.stage_node, &g.stage_params) != cudaSuccess) return false;
  g.stage_args.assign(g.stage_params.kernelParams, g.stage_params.kernelParams + g.stage_idx.count);
  if (cudaGraphInstantiate(&g.exec, graph, 0) != cudaSuccess) { g.exec = nullptr; return false; }
  g.graph = graph;                      // kept alive: the parameter blocks above belong to it
  return true;
}

static seg_status replay_graph(seg_handle* h, seg_handle::StepGraph& g, const void* x, const int32_t* cls,
                               float* loss_to, const float* gather) {
  if (x != g.cur_x || cls != g.cur_cls || gather != g.cur_gather || loss_to != g.cur_loss) {
    g.stage_args[g.stage_idx.x] = (void*)&x;
    g.stage_args[g.stage_idx.cls] = (void*)&cls;
    g.stage_args[g.stage_idx.gather] = (void*)&gather;
    g.stage_args[g.stage_idx.loss] = (void*)&loss_to;
    cudaKernelNodeParams sp = g.stage_params;
    sp.kernelParams = g.stage_args.data();
    SEG_TRY(h, cudaGraphExecKernelNodeSetParams(g.exec, g.stage_node, &sp), "graph parameter update");
    g.cur_x = x; g.cur_cls = cls; g.cur_gather = gather; g.cur_loss = loss_to;
  }
  SEG_TRY(h, cudaGraphLaunch(g.exec, h->stream), "graph launch");
  h->launches += g.kernels;
  for (int f = 0; f < FAM_COUNT; ++f) h->family_launches[f] += g.family[f];
  h->fused_updates += g.fused;
  if (g.peer) {
    g.peer->launches += g.kernels_peer;
    for (int f = 0; f < FAM_COUNT; ++f) g.peer->family_launches[f] += g.family_peer[f];
  }
  return SEG_OK;
}

// Runs one step through its captured graph: the first call with this graph slot runs eagerly (it sets
// kernel attributes), the second captures the same enqueue into a graph, later ones replay it with the
// caller's pointers written into the staging node.  enqueue(forked) enqueues the whole step; peer is a
// second handle whose kernels the step launches (the frozen right segment of a recovery step) or null.
static seg_status run_step_captured(seg_handle* h, seg_handle::StepGraph& g, seg_handle* peer,
                                    const std::function<seg_status(bool)>& enqueue,
                                    const void* x, const int32_t* cls, float* loss_to, const float* gather) {
  if (g.exec != nullptr) return replay_graph(h, g, x, cls, loss_to, gather);
  if (g.eager_runs == 0) {
    g.eager_runs = 1;
    return enqueue(h->fork_enabled);
  }
  const uint64_t before = h->launches, before_peer = peer ? peer->launches : 0;
  uint64_t fam_before[FAM_COUNT], fam_before_peer[FAM_COUNT] = {0, 0, 0, 0};
  for (int f = 0; f < FAM_COUNT; ++f) { fam_before[f] = h->family_launches[f]; if (peer) fam_before_peer[f] = peer->family_launches[f]; }
  const uint64_t fused_before = h->fused_updates;
  auto restore_counts = [&] {          // what a capture "launched" has not run: take it off the counters again
    h->launches = before;
    h->fused_updates = fused_before;
    for (int f = 0; f < FAM_COUNT; ++f) h->family_launches[f] = fam_before[f];
    if (peer) {
      peer->launches = before_peer;
      for (int f = 0; f < FAM_COUNT; ++f) peer->family_launches[f] = fam_before_peer[f];
    }
  };
  cudaGraph_t graph = nullptr;
  if (cudaStreamBeginCapture(h->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();
    h->graphs_enabled = false;
    return enqueue(h->fork_enabled);
  }
  h->capturing = true; h->cap_stage_node = nullptr;
  seg_status st = enqueue(h->fork_enabled);
  h->capturing = false;
  cudaError_t e = cudaStreamEndCapture(h->stream, &graph);
  if (st == SEG_OK && e == cudaSuccess && graph != nullptr && adopt_captured_graph(h, g, graph)) {
    g.kernels = h->launches - before;
    for (int f = 0; f < FAM_COUNT; ++f) g.family[f] = h->family_launches[f] - fam_before[f];
    g.fused = h->fused_updates - fused_before;
    g.peer = peer;
    if (peer) {
      g.kernels_peer = peer->launches - before_peer;
      for (int f = 0; f < FAM_COUNT; ++f) g.family_peer[f] = peer->family_launches[f] - fam_before_peer[f];
    }
    restore_counts();
    return replay_graph(h, g, x, cls, loss_to, gather);
  }
  // capture did not work here: run eagerly from now on
  if (getenv("SEG_DEBUG"))
    fprintf(stderr, "seg: step capture failed (status %d, end-capture '%s', node %p, last '%s')\n", (int)st,
            cudaGetErrorString(e), (void*)h->cap_stage_node, cudaGetErrorString(cudaPeekAtLastError()));
  cudaGetLastError();
  if (graph) cudaGraphDestroy(graph);
  g.exec = nullptr;
  h->graphs_enabled = false;
  restore_counts();
  return enqueue(h->fork_enabled);
}

static seg_status train_step_impl(seg_handle* h, const void* x, const int32_t* cls, int32_t batch,
                                  float* loss_out, void* y_out, const float* gather);

seg_status seg_train_step(seg_handle* h, const void* x, const int32_t* cls, int32_t batch,
                          float* loss_out, void* y_out) {
  if (!h || !x || !cls) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  return train_step_impl(h, x, cls, batch, loss_out, y_out, nullptr);
}

// Fully separate variant (Section 2, last flowchart): the segment's input is the intermediate label of the
// previous cut, gathered by class inside the staging kernel.
seg_status seg_train_step_label_input(seg_handle* h, const float* sil_in, const int32_t* cls, int32_t batch,
                                      float* loss_out) {
  if (!h || !sil_in || !cls) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  return train_step_impl(h, nullptr, cls, batch, loss_out, nullptr, sil_in);
}

static seg_status train_step_impl(seg_handle* h, const void* x, const int32_t* cls, int32_t batch,
                                  float* loss_out, void* y_out, const float* gather) {
  if (batch < 1 || batch > h->max_batch) return SEG_ERR_SHAPE;
  if (!h->is_final && !h->have_labels) return SEG_ERR_STATE;
  seg_status st = SEG_OK;
  if (h->profile || !h->graphs_enabled) {
    st = enqueue_step(h, batch, !h->profile && h->fork_enabled, x, cls, loss_out, gather);
  } else {
    auto enqueue = [&](bool forked) { return enqueue_step(h, batch, forked, x, cls, loss_out, gather); };
    st = run_step_captured(h, h->graphs[batch], nullptr, enqueue, x, cls, loss_out ? loss_out : h->loss_slot, gather);
  }
  if (st != SEG_OK) return st;
  ++h->step;
  h->last_batch = batch;           // a replayed graph does not pass through forward_layers
  if (y_out && (st = copy_out(h, y_out, batch)) != SEG_OK) return st;
  return SEG_OK;
}

// Recovery step (Section 5 of the paper): the left segment keeps training through the frozen right one.
static seg_status enqueue_recovery(seg_handle* h, seg_handle* r, int batch, bool forked, const void* x,
                                   const int32_t* cls, float* loss_to) {
  const int Ll = h->n_layers, Lr = r->n_layers;
  cudaStream_t s = h->stream;
  seg_status st;
  {
    Launch lc(h, K_COPY);
    SEG_TRY(h, launch_stage_inputs(h->x_stage, h->act_dt, h->ld_act[0], x, h->widths[0], batch, h->widths[0],
                                   h->act_round, h->cls_stage, cls, h->step_dev, h->bc_dev, h->beta1, h->beta2,
                                   nullptr, loss_to, h->loss_dst, h->n_classes, h->dev_status, s), "input staging");
  }
  if (h->capturing) { h->cap_stage_node = last_captured_node(h); h->cap_stage_idx = kStageInputsArgs; }
  if ((st = forward_layers(h, h->x_stage, h->ld_act[0], batch)) != SEG_OK) return st;
  // the joined network's loss: the right segment's softmax cross-entropy on the class labels
  if ((st = forward_layers(r, h->act[Ll], h->ld_act[Ll], batch, h->cls_stage, h->loss_dst)) != SEG_OK) return st;
  // through the frozen right segment: dgrad only, down to its input, which is the left segment's output
  for (int l = Lr - 1; l >= 0; --l) {
    const LayerInfo& Ly = r->layers[l];
    GemmDesc d{};
    d.A = r->dzbuf[l]; d.a_sm = r->ld_act[l + 1]; d.a_sk = 1; d.a_dt = r->act_dt;
    d.B = weights_op(r, l); d.b_sk = Ly.ldw; d.b_sn = 1; d.b_dt = r->op_dt;
    d.M = batch; d.N = Ly.in; d.K = Ly.out; d.c_dt = r->act_dt; d.c_round = r->act_round;
    if (l > 0) {
      d.C = r->dzbuf[l - 1]; d.ldc = r->ld_act[l];
      d.epi = EPI_MASK; d.mask = r->act[l]; d.ldmask = r->ld_act[l];
    } else {
      d.C = h->dzbuf[Ll - 1]; d.ldc = h->ld_act[Ll];
      if (h->last_relu) { d.epi = EPI_MASK; d.mask = h->act[Ll]; d.ldmask = h->ld_act[Ll]; }
      else d.epi = EPI_PLAIN;
    }
    if ((st = run_gemm(r, d, K_DGRAD, s)) != SEG_OK) return st;
  }
  return enqueue_backward(h, batch, forked);
}

seg_status seg_recovery_step(seg_handle* left, seg_handle* right, const void* x, const int32_t* cls,
                             int32_t batch, float* loss_out) {
  if (!left || !right || !x || !cls) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(left);
  if (left->device != right->device) return SEG_ERR_UNSUPPORTED;    // the joined network runs on one device
  if (batch < 1 || batch > left->max_batch || batch > right->max_batch) return SEG_ERR_SHAPE;
  if (left->is_final || !right->is_final) return SEG_ERR_STATE;
  if (left->widths[left->n_layers] != right->widths[0]) return SEG_ERR_SHAPE;
  if (left->precision != right->precision || left->stream != right->stream) return SEG_ERR_UNSUPPORTED;
  seg_handle* h = left;
  seg_handle* r = right;
  float* loss_to = loss_out ? loss_out : r->loss_slot;
  seg_status st;
  if (h->profile || r->profile || !h->graphs_enabled) {
    st = enqueue_recovery(h, r, batch, !h->profile && !r->profile && h->fork_enabled, x, cls, loss_to);
  } else {
    // captured like an ordinary step; the graph holds the right segment's buffers, so it is keyed by that
    // segment's identity and dropped with the left handle
    auto enqueue = [&](bool forked) { return enqueue_recovery(h, r, batch, forked, x, cls, loss_to); };
    st = run_step_captured(h, h->recovery_graphs[std::make_pair(r->uid, (int)batch)], r, enqueue, x, cls, loss_to, nullptr);
  }
  if (st != SEG_OK) return st;
  ++h->step;
  h->last_batch = r->last_batch = batch;
  return SEG_OK;
}

seg_status seg_train_epochs(seg_handle* h, const void* x, const int32_t* cls, int64_t n, int32_t batch,
                            int32_t epochs, float* losses) {
  if (!h || !x || !cls) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (n < 1 || epochs < 0) return SEG_ERR_SHAPE;
  if (batch < 1 || batch > h->max_batch) return SEG_ERR_SHAPE;
  const size_t row_bytes = (size_t)h->widths[0] * elem_size(h->act_dt);
  int64_t step = 0;
  for (int e = 0; e < epochs; ++e) {
    for (int64_t i = 0; i < n; i += batch, ++step) {
      const int b = (int)std::min<int64_t>(batch, n - i);
      seg_status st = seg_train_step(h, reinterpret_cast<const char*>(x) + (size_t)i * row_bytes, cls + i, b,
                                     losses ? losses + step : nullptr, nullptr);
      if (st != SEG_OK) return st;
    }
  }
  return SEG_OK;
}

seg_status seg_forward_dataset(seg_handle* h, const void* x, int64_t n, int32_t batch, void* y) {
  if (!h || !x || !y) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (n < 1) return SEG_ERR_SHAPE;
  if (batch < 1 || batch > h->max_batch) return SEG_ERR_SHAPE;
  const size_t in_bytes = (size_t)h->widths[0] * elem_size(h->act_dt);
  const size_t out_bytes = (size_t)h->widths[h->n_layers] * elem_size(h->act_dtype[h->n_layers]);
  for (int64_t i = 0; i < n; i += batch) {
    const int b = (int)std::min<int64_t>(batch, n - i);
    seg_status st = seg_forward(h, reinterpret_cast<const char*>(x) + (size_t)i * in_bytes, b,
                                reinterpret_cast<char*>(y) + (size_t)i * out_bytes);
    if (st != SEG_OK) return st;
  }
  return SEG_OK;
}

// Device-side address of a page-locked, mapped host buffer (what cudaHostAlloc, cudaHostRegister and
// torch's pinned tensors give); nullptr for pageable memory.
static const void* mapped_device_pointer(const void* host) {
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, host) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  if (a.type != cudaMemoryTypeHost || a.devicePointer == nullptr) return nullptr;
  return a.devicePointer;
}

seg_status seg_train_step_host(seg_handle* h, const void* x_host, const int32_t* cls_host, int32_t batch,
                               float* loss_host) {
  if (!h || !x_host || !cls_host) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (batch < 1 || batch > h->max_batch) return SEG_ERR_SHAPE;
  seg_status st;
  const size_t row_bytes = (size_t)h->widths[0] * elem_size(h->act_dt);
  // Page-locked batches are read by the staging kernel straight from host memory (the transfer happens
  // inside that kernel, no separate copy is enqueued); pageable ones go through a device buffer.
  const void* x_dev = mapped_device_pointer(x_host);
  const int32_t* cls_dev = reinterpret_cast<const int32_t*>(mapped_device_pointer(cls_host));
  if ((!x_dev || !cls_dev) && !h->host_x) {
    char* p = nullptr;
    if ((st = dev_alloc(h, &p, (size_t)h->max_batch * row_bytes, false)) != SEG_OK) return st;
    h->host_x = p;
    if ((st = dev_alloc(h, &h->host_cls, h->max_batch, false)) != SEG_OK) return st;
  }
  if (!h->host_loss) {
    // the loss lands in page-locked host memory the kernel writes directly: no copy back, one synchronisation
    void* p = nullptr;
    SEG_TRY(h, cudaHostAlloc(&p, sizeof(float), cudaHostAllocMapped), "page-locked loss slot");
    h->host_loss = reinterpret_cast<float*>(p);
    void* d = nullptr;
    SEG_TRY(h, cudaHostGetDevicePointer(&d, p, 0), "page-locked loss slot");
    h->host_loss_dev = reinterpret_cast<float*>(d);
  }
  if (!x_dev) {
    SEG_TRY(h, cudaMemcpyAsync(h->host_x, x_host, batch * row_bytes, cudaMemcpyHostToDevice, h->stream), "input copy");
    x_dev = h->host_x;
  }
  if (!cls_dev) {
    SEG_TRY(h, cudaMemcpyAsync(h->host_cls, cls_host, sizeof(int32_t) * batch, cudaMemcpyHostToDevice, h->stream), "class copy");
    cls_dev = h->host_cls;
  }
  if ((st = seg_train_step(h, x_dev, cls_dev, batch, h->host_loss_dev, nullptr)) != SEG_OK) return st;
  SEG_TRY(h, cudaStreamSynchronize(h->stream), "stream synchronize");
  if (loss_host) *loss_host = *reinterpret_cast<volatile float*>(h->host_loss);
  return SEG_OK;
}

seg_status seg_train_step_host_async(seg_handle* h, const void* x_host, const int32_t* cls_host, int32_t batch,
                                     float* loss_host) {
  if (!h || !x_host || !cls_host) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (batch < 1 || batch > h->max_batch) return SEG_ERR_SHAPE;
  if (!mapped_device_pointer(x_host) || !mapped_device_pointer(cls_host)) return SEG_ERR_INVALID_ARG;   // pageable
  float* loss_dev = nullptr;
  if (loss_host) {
    loss_dev = reinterpret_cast<float*>(const_cast<void*>(mapped_device_pointer(loss_host)));
    if (!loss_dev) return SEG_ERR_INVALID_ARG;
  }
  // The batch travels on a copy stream into one of two device buffers, so that the transfer of this
  // step's batch overlaps the kernels of the steps enqueued before it; the step waits for its copy, and a
  // buffer is overwritten only after the step that last read it is complete.
  seg_status st;
  const size_t row_bytes = (size_t)h->widths[0] * elem_size(h->act_dt);
  if (!h->copy_stream) {
    SEG_TRY(h, cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking), "copy stream");
    for (int i = 0; i < 2; ++i) {
      char* p = nullptr;
      if ((st = dev_alloc(h, &p, (size_t)h->max_batch * row_bytes, false)) != SEG_OK) return st;
      h->async_x[i] = p;
      if ((st = dev_alloc(h, &h->async_cls[i], h->max_batch, false)) != SEG_OK) return st;
      SEG_TRY(h, cudaEventCreateWithFlags(&h->ev_copied[i], cudaEventDisableTiming), "event create");
      SEG_TRY(h, cudaEventCreateWithFlags(&h->ev_consumed[i], cudaEventDisableTiming), "event create");
    }
  }
  const int i = h->async_next;
  h->async_next ^= 1;
  if (h->async_used[i]) SEG_TRY(h, cudaStreamWaitEvent(h->copy_stream, h->ev_consumed[i], 0), "stream wait");
  SEG_TRY(h, cudaMemcpyAsync(h->async_x[i], x_host, batch * row_bytes, cudaMemcpyHostToDevice, h->copy_stream), "input copy");
  SEG_TRY(h, cudaMemcpyAsync(h->async_cls[i], cls_host, sizeof(int32_t) * batch, cudaMemcpyHostToDevice, h->copy_stream), "class copy");
  SEG_TRY(h, cudaEventRecord(h->ev_copied[i], h->copy_stream), "event record");
  SEG_TRY(h, cudaStreamWaitEvent(h->stream, h->ev_copied[i], 0), "stream wait");
  if ((st = seg_train_step(h, h->async_x[i], h->async_cls[i], batch, loss_dev, nullptr)) != SEG_OK) return st;
  SEG_TRY(h, cudaEventRecord(h->ev_consumed[i], h->stream), "event record");
  h->async_used[i] = true;
  return SEG_OK;
}

seg_status seg_get_labels(seg_handle* h, float* dst) {
  if (!h || !dst) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (h->is_final || !h->have_labels) return SEG_ERR_STATE;
  SEG_TRY(h, cudaMemcpyAsync(dst, h->sil, sizeof(float) * h->n_classes * h->widths[h->n_layers],
                             cudaMemcpyDeviceToDevice, h->stream), "label copy");
  return SEG_OK;
}

seg_status seg_set_labels(seg_handle* h, const float* src) {
  if (!h || !src) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (h->is_final) return SEG_ERR_STATE;
  SEG_TRY(h, cudaMemcpyAsync(h->sil, src, sizeof(float) * h->n_classes * h->widths[h->n_layers],
                             cudaMemcpyDeviceToDevice, h->stream), "label copy");
  h->have_labels = true;
  return SEG_OK;
}

static seg_status get_flat(seg_handle* h, const float* base, int layer, float* W, float* b) {
  if (!h) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (!valid_layer(h, layer)) return SEG_ERR_SHAPE;
  if (!base) return SEG_ERR_STATE;
  const LayerInfo& L = h->layers[layer];
  if (W) {
    Launch l(h, K_COPY);
    SEG_TRY(h, launch_copy2d(W, DT_F32, L.in, base + L.w_off, DT_F32, L.ldw, L.out, L.in, RND_NONE, h->stream), "tensor copy");
  }
  if (b) SEG_TRY(h, cudaMemcpyAsync(b, base + L.b_off, sizeof(float) * L.out, cudaMemcpyDeviceToDevice, h->stream), "tensor copy");
  return SEG_OK;
}

seg_status seg_get_params(seg_handle* h, int32_t layer, float* W, float* b) {
  return get_flat(h, h ? h->params : nullptr, layer, W, b);
}

seg_status seg_get_grads(seg_handle* h, int32_t layer, float* dW, float* db) {
  return get_flat(h, h ? h->grads : nullptr, layer, dW, db);
}

seg_status seg_get_opt_state(seg_handle* h, int32_t layer, int32_t which, float* sW, float* sb) {
  if (!h) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (which != 0 && which != 1) return SEG_ERR_INVALID_ARG;
  return get_flat(h, which == 0 ? h->state1 : h->state2, layer, sW, sb);
}

seg_status seg_set_opt_state(seg_handle* h, int32_t layer, int32_t which, const float* sW, const float* sb) {
  if (!h) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (which != 0 && which != 1) return SEG_ERR_INVALID_ARG;
  if (!valid_layer(h, layer)) return SEG_ERR_SHAPE;
  float* base = which == 0 ? h->state1 : h->state2;
  if (!base) return SEG_ERR_STATE;
  const LayerInfo& L = h->layers[layer];
  if (sW) {
    Launch l(h, K_COPY);
    SEG_TRY(h, launch_copy2d(base + L.w_off, DT_F32, L.ldw, sW, DT_F32, L.in, L.out, L.in, RND_NONE, h->stream), "tensor copy");
  }
  if (sb) SEG_TRY(h, cudaMemcpyAsync(base + L.b_off, sb, sizeof(float) * L.out, cudaMemcpyDeviceToDevice, h->stream), "tensor copy");
  return SEG_OK;
}

seg_status seg_get_step(const seg_handle* h, uint64_t* step) {
  if (!h || !step) return SEG_ERR_INVALID_ARG;
  *step = h->step;
  return SEG_OK;
}

seg_status seg_set_step(seg_handle* h, uint64_t step) {
  if (!h) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  h->step = step;
  const unsigned long long t = step;
  SEG_TRY(h, cudaMemcpyAsync(h->step_dev, &t, sizeof(t), cudaMemcpyHostToDevice, h->stream), "step counter copy");
  SEG_TRY(h, cudaStreamSynchronize(h->stream), "stream synchronize");
  return SEG_OK;
}

seg_status seg_set_params(seg_handle* h, int32_t layer, const float* W, const float* b) {
  if (!h) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (!valid_layer(h, layer)) return SEG_ERR_SHAPE;
  const LayerInfo& L = h->layers[layer];
  if (W) {
    Launch l(h, K_COPY);
    SEG_TRY(h, launch_copy2d(h->params + L.w_off, DT_F32, L.ldw, W, DT_F32, L.in, L.out, L.in, RND_NONE, h->stream), "tensor copy");
  }
  if (b) SEG_TRY(h, cudaMemcpyAsync(h->params + L.b_off, b, sizeof(float) * L.out, cudaMemcpyDeviceToDevice, h->stream), "tensor copy");
  const int64_t end = (layer + 1 < h->n_layers) ? h->layers[layer + 1].w_off : h->n_flat;
  return refresh_operand_copy(h, L.w_off, end - L.w_off);
}

seg_status seg_get_activation(seg_handle* h, int32_t layer, float* dst) {
  if (!h || !dst) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (layer < 1 || layer > h->n_layers) return SEG_ERR_SHAPE;
  if (h->last_batch < 1) return SEG_ERR_STATE;
  Launch l(h, K_COPY);
  SEG_TRY(h, launch_copy2d(dst, DT_F32, h->widths[layer], h->act[layer], h->act_dtype[layer], h->ld_act[layer],
                           h->last_batch, h->widths[layer], RND_NONE, h->stream), "activation copy");
  return SEG_OK;
}

seg_status seg_mem_bytes(const seg_handle* h, uint64_t* current, uint64_t* peak) {
  if (!h) return SEG_ERR_INVALID_ARG;
  if (current) *current = h->mem_current;
  if (peak) *peak = h->mem_peak;
  return SEG_OK;
}

seg_status seg_launch_count(const seg_handle* h, uint64_t* launches) {
  if (!h || !launches) return SEG_ERR_INVALID_ARG;
  *launches = h->launches;
  return SEG_OK;
}

seg_status seg_poll_status(seg_handle* h) {
  if (!h) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  int host = 0;
  SEG_TRY(h, cudaMemcpyAsync(&host, h->dev_status, sizeof(int), cudaMemcpyDeviceToHost, h->stream), "status read");
  SEG_TRY(h, cudaStreamSynchronize(h->stream), "stream synchronize");
  if (host != DEV_OK) {
    cudaMemsetAsync(h->dev_status, 0, sizeof(int), h->stream);
    if (host & DEV_TIMEOUT) {
      h->last_error = "a kernel gave up a bounded wait";
      return SEG_ERR_DEVICE_TIMEOUT;
    }
    h->last_error = "a step met a class index outside [0, n_classes); it was clamped";
    return SEG_ERR_CLASS_RANGE;
  }
  return SEG_OK;
}

seg_status seg_product_launches(const seg_handle* h, uint64_t* counts) {
  if (!h || !counts) return SEG_ERR_INVALID_ARG;
  for (int f = 0; f < FAM_COUNT; ++f) counts[f] = h->family_launches[f];
  counts[FAM_COUNT] = h->fused_updates;
  return SEG_OK;
}

seg_status seg_device(const seg_handle* h, int32_t* device) {
  if (!h || !device) return SEG_ERR_INVALID_ARG;
  *device = h->device;
  return SEG_OK;
}

seg_status seg_selftest_bounded_wait(seg_handle* h, uint64_t limit_ns) {
  if (!h) return SEG_ERR_INVALID_ARG;
  if (limit_ns < 1000ull || limit_ns > 1000000000ull) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  ++h->launches;
  SEG_TRY(h, launch_wait_selftest(h->dev_status, limit_ns, h->stream), "bounded-wait self-test");
  return SEG_OK;
}

// Section 2.1: the only data that ever moves between partitions is the stored response of the previous one.
seg_status seg_handoff_copy(seg_handle* producer, const void* src, seg_handle* consumer, void* dst, uint64_t bytes) {
  if (!producer || !consumer || !src || !dst) return SEG_ERR_INVALID_ARG;
  if (bytes == 0) return SEG_OK;
  seg_handle* h = producer;
  DeviceGuard guard(h);
  if (producer->device == consumer->device) {
    SEG_TRY(h, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, producer->stream), "hand-off copy");
  } else {
    SEG_TRY(h, cudaMemcpyPeerAsync(dst, consumer->device, src, producer->device, bytes, producer->stream), "hand-off copy");
  }
  if (producer->stream == consumer->stream) return SEG_OK;     // one stream: already ordered
  if (!producer->ev_handoff)
    SEG_TRY(h, cudaEventCreateWithFlags(&producer->ev_handoff, cudaEventDisableTiming), "event create");
  SEG_TRY(h, cudaEventRecord(producer->ev_handoff, producer->stream), "event record");
  DeviceGuard guard_consumer(consumer);
  SEG_TRY(consumer, cudaStreamWaitEvent(consumer->stream, producer->ev_handoff, 0), "stream wait");
  return SEG_OK;
}

seg_status seg_timer_start(seg_handle* h) {
  if (!h) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  SEG_TRY(h, cudaEventRecord(h->ev_start, h->stream), "event record");
  return SEG_OK;
}

seg_status seg_timer_stop(seg_handle* h) {
  if (!h) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  SEG_TRY(h, cudaEventRecord(h->ev_stop, h->stream), "event record");
  return SEG_OK;
}

seg_status seg_timer_elapsed_ms(seg_handle* h, float* ms) {
  if (!h || !ms) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  SEG_TRY(h, cudaEventSynchronize(h->ev_stop), "event synchronize");
  SEG_TRY(h, cudaEventElapsedTime(ms, h->ev_start, h->ev_stop), "event elapsed");
  return SEG_OK;
}

seg_status seg_profile_enable(seg_handle* h, int32_t on) {
  if (!h) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  SEG_TRY(h, cudaStreamSynchronize(h->stream), "stream synchronize");
  h->profile = on != 0;
  h->ev_used = 0;
  h->ev_kind.clear();
  return SEG_OK;
}

seg_status seg_profile_get(seg_handle* h, int32_t kind, uint64_t* count, float* total_ms) {
  if (!h || !count || !total_ms) return SEG_ERR_INVALID_ARG;
  DeviceGuard guard(h);
  if (kind < 0 || kind >= K_COUNT) return SEG_ERR_INVALID_ARG;
  SEG_TRY(h, cudaStreamSynchronize(h->stream), "stream synchronize");
  uint64_t n = 0; double total = 0.0;
  for (size_t i = 0; i < h->ev_kind.size() && 2 * i + 1 < h->ev_used; ++i) {
    if (h->ev_kind[i] != kind) continue;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, h->ev_pool[2 * i], h->ev_pool[2 * i + 1]) == cudaSuccess) { total += ms; ++n; }
  }
  *count = n; *total_ms = (float)total;
  return SEG_OK;
}

}  // extern "C"
