// Shared declarations of the segment-trainer library (internal; the public ABI is include/seg.h).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "seg.h"

namespace segk {

// Storage type of an operand / activation buffer.
enum DType : int { DT_F32 = 0, DT_BF16 = 1 };
// Rounding applied when a value is stored into a buffer that later feeds a matrix product.
enum Round : int { RND_NONE = 0, RND_TF32 = 1, RND_BF16 = 2 };

// Epilogues of the three matrix products of a Linear layer.
enum Epilogue : int {
  EPI_BIAS_ACT = 0,  // forward: + bias[n], optional ReLU
  EPI_MASK = 1,      // dgrad:   * (mask[m][n] > 0)  (mask = stored post-ReLU activation)
  EPI_PLAIN = 2      // wgrad:   store the fp32 product
};

// Device status word: bits OR-ed in by kernels (a bounded wait that ran out; a class index outside
// [0, M) met and clamped by the input staging).
enum DevStatus : int { DEV_OK = 0, DEV_TIMEOUT = 1, DEV_BAD_CLASS = 2 };

// Families of matrix-product kernels (reported per handle by seg_product_launches).
enum Family : int { FAM_TC_SINGLE = 0, FAM_TC_SPLITK = 1, FAM_TC_PAIR = 2, FAM_SIMT = 3, FAM_COUNT = 4 };

// The loss of a non-final segment fused into the epilogue of its last forward product when the
// split-K kernel runs it (Section 2: the target is the intermediate label of the sample's class; the
// final segment's softmax cross-entropy always runs as a launch of its own).  The epilogue still
// stores the layer's output; in addition it writes dZ of that layer and adds up the batch loss (one
// partial per CTA; the last CTA to finish adds the partials in index order, writes the loss to the
// address found in *loss_dst and leaves the counter at zero).
struct LossFuse {
  int enabled;              // 0: no fused loss
  const int32_t* cls;       // [M]: class index of every row
  const float* sil;         // [classes][N] fp32 targets
  void* dz;                 // [M][ld_dz] of dz_dt, rounded by dz_round
  int64_t ld_dz;
  int dz_dt, dz_round;
  int relu_mask;            // dZ = 0 where the stored output is not positive
  float gscale;             // dZ factor: 2/(M N)
  float loss_scale;         // factor of the summed loss: 1/(M N)
  float* partials;          // one float per CTA of the launch
  unsigned int* counter;    // arrival counter, zero between launches
  float* const* loss_dst;   // device slot holding the address that receives the loss
};

// The optimizer update of a layer's weights applied inside its weight-gradient product (tensor-core
// persistent kernels only, opt-in: it measured slower than the separate update launch): extra warps
// of every CTA stream over each output tile once the epilogue warps have stored it, so that the
// update's HBM traffic runs under the main loop of the following tiles instead of after the product.
// All pointers address the layer's weight tensor, laid out as the product's C: element (m, n) at
// base + m * ldc + n.
struct FusedUpdate {
  int enabled;              // 0: plain product
  float* p;                 // fp32 master weights
  float* s1;                // momentum buffer / Adam first moment (null for plain SGD)
  float* s2;                // Adam second moment (null otherwise)
  void* p_op;               // reduced-precision operand copy of the weights (never null on this path)
  int op_dt, op_round;      // DType / Round of p_op
  int optimizer;            // seg_optimizer
  float lr, momentum, beta1, beta2, eps;
  const float* bc;          // device: {1-b1^t, 1-b2^t}
};

// One matrix product  C[M][N] = sum_k A(m,k) * B(k,n)  with explicit element strides, so that
// forward (A W^T), dgrad (dZ W) and wgrad (dZ^T A) are all expressed by one description.
struct GemmDesc {
  const void* A;   // element (m,k) at A + m*a_sm + k*a_sk   (elements of a_dt)
  const void* B;   // element (k,n) at B + k*b_sk + n*b_sn   (elements of b_dt)
  void* C;         // element (m,n) at C + m*ldc + n         (elements of c_dt)
  int64_t a_sm, a_sk, b_sk, b_sn, ldc;
  int M, N, K;
  int a_dt, b_dt, c_dt;     // DType
  int c_round;              // Round applied to C on store
  int epi;                  // Epilogue
  int relu;                 // EPI_BIAS_ACT: apply ReLU
  const float* bias;        // EPI_BIAS_ACT: [N]
  const void* mask;         // EPI_MASK: [M][ldmask] of c_dt
  int64_t ldmask;
  LossFuse loss;            // EPI_BIAS_ACT only
  FusedUpdate upd;          // EPI_PLAIN (weight gradient) only
  int off_critical_path;    // 1: the product runs beside others (a weight gradient on its branch): the tiling is
                            // chosen for latency plus the SM time it takes away from them, not for latency alone
  // FFMA path only: workspace for splitting K over several CTAs of one tile (may be null: no split).
  // simt_scratch holds simt_slots partial tiles of 64 x 64 floats, simt_counters one arrival counter
  // per slot (zero between launches).  Products that may run at the same time need separate workspaces.
  float* simt_scratch;
  unsigned int* simt_counters;
  int simt_slots;
};
constexpr int kSimtTileFloats = 64 * 64;

// ---- launchers (each returns the cudaError_t of its launch) -------------------------------
cudaError_t launch_gemm_simt(const GemmDesc& g, cudaStream_t s);
int gemm_simt_slots(int M, int N, int K);   // workspace slots (partial 64 x 64 tiles) a split of this product would use
// Tensor-core path.  Returns cudaErrorNotSupported when the shape/stride does not fit its TMA rules.
// *family (may be null) receives the Family of the kernel that was launched.
cudaError_t launch_gemm_tc(const GemmDesc& g, int* dev_status, cudaStream_t s, int* family = nullptr);
bool gemm_tc_init();   // resolves the driver entry point needed for tensor maps (once per process, thread-safe)
// One block that waits, with the product kernels' bounded wait, on a barrier nothing arrives at.
cudaError_t launch_wait_selftest(int* dev_status, uint64_t limit_ns, cudaStream_t s);
// True when launch_gemm_tc would take the intermediate-label loss into the forward product M x N x K.
bool gemm_tc_can_fuse_loss(int M, int N, int K, bool tf32);
// True when launch_gemm_tc would run this weight-gradient product (both operands MN-major, EPI_PLAIN) in a
// persistent kernel that can apply the optimizer update as well (g.upd is not looked at).
bool gemm_tc_can_fuse_update(const GemmDesc& g);

cudaError_t launch_gen_labels(float* dst, int n_classes, int n_p, uint64_t seed, int segment_id,
                              int dist, float kappa, cudaStream_t s);
cudaError_t launch_init_uniform(float* dst, int rows, int cols, int64_t ld, uint64_t seed,
                                int segment_id, int layer, int tag, float bound, cudaStream_t s);

// loss kernels: write dZ (dz_dt, rounded by dz_round) and a deterministic batch loss, which goes to
// the address stored in the device slot *loss_dst (the input-staging launch of the step fills it)
cudaError_t launch_mse_loss(const void* out, int out_dt, int64_t ld_out, const int32_t* cls,
                            const float* sil, int n_classes, int n_p, int batch, int relu_mask,
                            void* dz, int dz_dt, int dz_round, int64_t ld_dz,
                            float* partials, unsigned int* counter, float* const* loss_dst, cudaStream_t s);
cudaError_t launch_softmax_ce_loss(const float* logits, int64_t ld_logits, const int32_t* cls,
                                   int n_classes, int batch, int relu_mask,
                                   void* dz, int dz_dt, int dz_round, int64_t ld_dz,
                                   float* partials, unsigned int* counter, float* const* loss_dst,
                                   cudaStream_t s);
int loss_max_partials();

// One layer's update.  p, g, s1, s2, p_op point at the layer's weight tensor in the flat ranges; n
// elements from there are streamed (the weight tensor with its zero padding).  When dz is not null
// the launch also forms the bias gradient g_bias[c] = sum_b dz[b][c], c < n_bias, and updates the
// n_bias bias elements that start bias_off elements after p.
struct UpdateArgs {
  float* p; const float* g; float* s1; float* s2;
  void* p_op;          // reduced-precision operand copy (may be null)
  int op_dt;           // DType of p_op
  int op_round;        // Round for p_op
  int64_t n;
  const void* dz;      // [batch][ld_dz] of dz_dt: dZ of this layer (may be null: no bias part)
  int dz_dt;
  int64_t ld_dz;
  int batch, n_bias;
  int64_t bias_off;
  float* g_bias;       // [n_bias]: receives the bias gradient
  int optimizer;
  float lr, momentum, beta1, beta2, eps;
  const float* bc;     // device: {1-b1^t, 1-b2^t}, Adam's bias corrections for this step
};
cudaError_t launch_update(const UpdateArgs& u, cudaStream_t s);

// copies with pitch / dtype / rounding conversion: dst[r][c] = cvt(src[r][c])
cudaError_t launch_copy2d(void* dst, int dst_dt, int64_t ld_dst, const void* src, int src_dt,
                          int64_t ld_src, int64_t rows, int64_t cols, int round, cudaStream_t s);
// the same copy plus an int32 vector copy (class indices) in one launch; when t is not null the
// launch also advances the step counter: t += 1, bc = {1 - beta1^t, 1 - beta2^t}; when gather_src is not
// null, row r of the destination is row cls[r] of that fp32 [classes][cols] matrix instead of src's row r;
// when loss_dst is not null the launch stores loss_out there (the step's loss kernel reads it back).
// Class indices are clamped to [0, n_classes) on the way; one outside sets DEV_BAD_CLASS in *dev_status.
cudaError_t launch_stage_inputs(void* dst, int dt, int64_t ld_dst, const void* src, int64_t ld_src, int rows,
                                int cols, int round, int32_t* cls_dst, const int32_t* cls_src,
                                unsigned long long* t, float* bc, float beta1, float beta2,
                                const float* gather_src, float* loss_out, float** loss_dst,
                                int n_classes, int* dev_status, cudaStream_t s);

// ---- programmatic dependent launch ------------------------------------------------------------
// Kernels of one stream are launched with programmatic stream serialisation: a kernel may become
// resident and run its prologue while its predecessor drains.  Every kernel therefore calls
// pdl_wait() before its first access to global memory (it returns once the predecessor grid has
// completed and its writes are visible; a no-op for ordinary launches) and pdl_trigger() to let its
// own successor start early.
extern bool g_use_pdl;
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                            Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = g_use_pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// ---- optimizer step on one element ------------------------------------------------------------
// Section 3: SGD with momentum; plain SGD and Adam as well.  H supplies lr, momentum, beta1, beta2, eps.
template <int OPT, typename H>
__device__ __forceinline__ void opt_step(float& p, float g, float& m, float& v, const H& u,
                                         float inv_bc1, float inv_bc2) {
  if constexpr (OPT == SEG_SGD) {
    p = p - u.lr * g;
  } else if constexpr (OPT == SEG_SGD_MOMENTUM) {
    m = u.momentum * m + g;
    p = p - u.lr * m;
  } else {
    m = u.beta1 * m + (1.0f - u.beta1) * g;
    v = u.beta2 * v + (1.0f - u.beta2) * g * g;
    const float mhat = m * inv_bc1;
    const float vhat = v * inv_bc2;
    p = p - u.lr * mhat / (sqrtf(vhat) + u.eps);
  }
}

// ---- small device helpers ------------------------------------------------------------------
__device__ __forceinline__ float round_tf32_rne(float x) {
  uint32_t u = __float_as_uint(x);
  u = (u + 0x0FFFu + ((u >> 13) & 1u)) & 0xFFFFE000u;
  return __uint_as_float(u);
}
__device__ __forceinline__ float round_bf16_rne(float x) {
  return __bfloat162float(__float2bfloat16_rn(x));
}
__device__ __forceinline__ float apply_round(float x, int mode) {
  if (mode == RND_TF32) return round_tf32_rne(x);
  if (mode == RND_BF16) return round_bf16_rne(x);
  return x;
}
__device__ __forceinline__ float load_as_float(const void* p, int dt, int64_t i) {
  return dt == DT_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i])
                       : reinterpret_cast<const float*>(p)[i];
}
__device__ __forceinline__ void store_from_float(void* p, int dt, int64_t i, float v) {
  if (dt == DT_BF16) reinterpret_cast<__nv_bfloat16*>(p)[i] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(p)[i] = v;
}

// ---- whole step of a small fp32 segment in two launches ---------------------------------------------
// A segment of at most kSmallMaxLayers layers, none wider than kSmallMaxWidth, fed kSmallMaxInput features at
// most (Section 3: 784-80-60 and 60-60-60-47) is latency-bound when every product, the loss and every update
// is a launch of its own.  The first kernel carries a slice of the batch through staging, all forward
// products, the loss and the dgrad chain; the second forms every layer's weight and bias gradient and
// applies the optimizer.  Description of one step for both (all pointers device, fp32):
constexpr int kSmallMaxLayers = 4, kSmallMaxWidth = 128, kSmallMaxInput = 1024;
struct SmallStep {
  int n_layers, batch, n_classes, is_final, last_relu, optimizer;
  int widths[kSmallMaxLayers + 1];
  int64_t ldw[kSmallMaxLayers], w_off[kSmallMaxLayers], b_off[kSmallMaxLayers];   // element offsets into the flat ranges
  int64_t ld_act[kSmallMaxLayers + 1];
  float* params; float* grads; float* s1; float* s2;
  float* act[kSmallMaxLayers + 1];     // act[0]: the staged input
  float* dz[kSmallMaxLayers];
  const float* sil;
  int32_t* cls_stage;
  float* loss_partials; unsigned int* loss_counter; float** loss_dst;
  unsigned long long* t; float* bc;
  int* dev_status;
  float lr, momentum, beta1, beta2, eps;
  float* wg_scratch; unsigned int* wg_counters; int wg_slots;   // partial 64 x 64 tiles of the weight-gradient kernel
};
bool small_step_supported(int n_layers, const int* widths);   // the shape limits above
bool small_step_batch_ok(int batch);                          // one loss partial per CTA: bounded by loss_max_partials()
int small_step_wgrad_slots(int n_layers, const int* widths);  // partial tiles (and counters) the second kernel may use
cudaError_t launch_small_fwd_bwd(const SmallStep& p, const float* x, const int32_t* cls, const float* gather,
                                 float* loss_to, cudaStream_t s);
cudaError_t launch_small_wgrad_update(const SmallStep& p, cudaStream_t s);

// ---- reductions -------------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}
// Sum over the block in a fixed order (deterministic for a fixed launch shape); valid in warp 0.
__device__ inline float block_sum(float v, float* smem /* >= 32 floats */) {
  v = warp_sum(v);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __syncthreads();
  if (lane == 0) smem[warp] = v;
  __syncthreads();
  float total = 0.f;
  if (warp == 0) {
    const int n_warps = (blockDim.x + 31) >> 5;
    total = lane < n_warps ? smem[lane] : 0.f;
    total = warp_sum(total);
  }
  return total;
}
// Writes this block's partial; the last block to finish adds all partials in index order and
// writes scale * total to loss_out, or, when loss_dst is not null, to the address stored in
// *loss_dst.  The counter is left at zero for the next launch.
__device__ inline void finish_loss(float block_total, float* partials, unsigned int* counter,
                            float* loss_out, float* const* loss_dst, float scale, float* smem) {
  __shared__ bool is_last;
  if (threadIdx.x == 0) {
    partials[blockIdx.x] = block_total;
    __threadfence();
    const unsigned int done = atomicAdd(counter, 1u);
    is_last = (done == gridDim.x - 1);
  }
  __syncthreads();
  if (is_last) {
    __threadfence();
    float v = 0.f;
    for (int i = threadIdx.x; i < (int)gridDim.x; i += blockDim.x) v += __ldcg(partials + i);
    const float total = block_sum(v, smem);
    if (threadIdx.x == 0) {
      if (loss_dst) loss_out = *loss_dst;
      if (loss_out) *loss_out = total * scale;
      *counter = 0u;
    }
  }
}

}  // namespace segk
