// Streaming kernels of the segment step: the two losses (Section 2: intermediate-label
// regression for a non-final segment, class labels for the final one), the optimizer update
// with the bias gradient formed in the same launch (Section 3: SGD with momentum; plain SGD and Adam as well) and
// pitch/dtype conversion copies.  All of them are HBM-bound; none uses tensor cores.
#include "common.cuh"

namespace segk {

bool g_use_pdl = true;

namespace {

constexpr int kLossThreads = 256;
constexpr int kMaxLossBlocks = 1024;

// Non-final segment: target of sample b is row cls[b] of the label matrix (gathered here, never
// materialised per sample);  loss = mean (a - t)^2,  dZ = 2 (a - t) / (B N_P) * [a > 0].
// A thread handles VEC consecutive columns of one row per pass (VEC = 8: 16-byte accesses for bf16,
// two for fp32 and for the fp32 targets); VEC = 1 serves widths that are not multiples of 8.  A class
// index outside [0, n_classes) is clamped, so that nothing is read out of bounds.
template <typename TOut, typename TDz, int VEC>
__global__ void __launch_bounds__(kLossThreads)
mse_loss_kernel(const TOut* __restrict__ out, int64_t ld_out, const int32_t* __restrict__ cls,
                const float* __restrict__ sil, int n_classes, int n_p, int batch, int relu_mask,
                TDz* __restrict__ dz, int dz_round, int64_t ld_dz, float* partials,
                unsigned int* counter, float* loss_out, float* const* loss_dst) {
  pdl_wait();
  pdl_trigger();
  __shared__ float red[32];
  const float gscale = 2.0f / (float)((int64_t)batch * n_p);
  float acc = 0.f;
  const unsigned int groups_per_row = (unsigned int)(n_p / VEC);
  const int64_t n_groups = (int64_t)batch * groups_per_row;
  for (int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; v < n_groups;
       v += (int64_t)gridDim.x * blockDim.x) {
    const int b = (int)(v / groups_per_row);
    const int i = (int)(v - (int64_t)b * groups_per_row) * VEC;
    const int c = min(max(__ldg(cls + b), 0), n_classes - 1);
    const float* trow = sil + (int64_t)c * n_p + i;
    float a[VEC], t[VEC], g[VEC];
    if constexpr (VEC == 8) {
      if constexpr (sizeof(TOut) == 2) {
        const uint4 q = *reinterpret_cast<const uint4*>(out + (int64_t)b * ld_out + i);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          a[2 * j] = __uint_as_float(w[j] << 16);
          a[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
        }
      } else {
        const float4 q0 = *reinterpret_cast<const float4*>(out + (int64_t)b * ld_out + i);
        const float4 q1 = *reinterpret_cast<const float4*>(out + (int64_t)b * ld_out + i + 4);
        a[0] = q0.x; a[1] = q0.y; a[2] = q0.z; a[3] = q0.w; a[4] = q1.x; a[5] = q1.y; a[6] = q1.z; a[7] = q1.w;
      }
      const float4 t0 = __ldg(reinterpret_cast<const float4*>(trow));
      const float4 t1 = __ldg(reinterpret_cast<const float4*>(trow + 4));
      t[0] = t0.x; t[1] = t0.y; t[2] = t0.z; t[3] = t0.w; t[4] = t1.x; t[5] = t1.y; t[6] = t1.z; t[7] = t1.w;
    } else {
      if constexpr (sizeof(TOut) == 2) a[0] = __bfloat162float(out[(int64_t)b * ld_out + i]);
      else a[0] = out[(int64_t)b * ld_out + i];
      t[0] = __ldg(trow);
    }
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
      const float d = a[j] - t[j];
      acc = fmaf(d, d, acc);
      float gj = d * gscale;
      if (relu_mask && !(a[j] > 0.f)) gj = 0.f;
      g[j] = apply_round(gj, dz_round);
    }
    if constexpr (VEC == 8) {
      if constexpr (sizeof(TDz) == 2) {
        uint4 q;
        __nv_bfloat162 p0 = __floats2bfloat162_rn(g[0], g[1]), p1 = __floats2bfloat162_rn(g[2], g[3]);
        __nv_bfloat162 p2 = __floats2bfloat162_rn(g[4], g[5]), p3 = __floats2bfloat162_rn(g[6], g[7]);
        q.x = *reinterpret_cast<uint32_t*>(&p0); q.y = *reinterpret_cast<uint32_t*>(&p1);
        q.z = *reinterpret_cast<uint32_t*>(&p2); q.w = *reinterpret_cast<uint32_t*>(&p3);
        *reinterpret_cast<uint4*>(dz + (int64_t)b * ld_dz + i) = q;
      } else {
        *reinterpret_cast<float4*>(dz + (int64_t)b * ld_dz + i) = make_float4(g[0], g[1], g[2], g[3]);
        *reinterpret_cast<float4*>(dz + (int64_t)b * ld_dz + i + 4) = make_float4(g[4], g[5], g[6], g[7]);
      }
    } else {
      if constexpr (sizeof(TDz) == 2) dz[(int64_t)b * ld_dz + i] = __float2bfloat16_rn(g[0]);
      else dz[(int64_t)b * ld_dz + i] = g[0];
    }
  }
  const float bt = block_sum(acc, red);
  finish_loss(bt, partials, counter, loss_out, loss_dst, 1.0f / (float)((int64_t)batch * n_p), red);
}

// Final segment: one warp per sample;  p = softmax(z) with the row maximum subtracted,
// loss = -mean log p[cls],  dZ = (p - onehot) / B.  Rows of up to 32 * CE_REGS classes are read once and kept
// in registers (lane i holds classes i, i + 32, ...); wider rows are read three times.
constexpr int CE_REGS = 32;
template <typename TDz, bool IN_REGS>
__global__ void __launch_bounds__(kLossThreads)
softmax_ce_kernel(const float* __restrict__ logits, int64_t ld, const int32_t* __restrict__ cls,
                  int n_classes, int batch, int relu_mask, TDz* __restrict__ dz, int dz_round,
                  int64_t ld_dz, float* partials, unsigned int* counter, float* loss_out,
                  float* const* loss_dst) {
  pdl_wait();
  pdl_trigger();
  __shared__ float red[32];
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  const float inv_b = 1.0f / (float)batch;
  float acc = 0.f;
  for (int b = blockIdx.x * warps_per_block + (threadIdx.x >> 5); b < batch;
       b += gridDim.x * warps_per_block) {
    const float* z = logits + (int64_t)b * ld;
    const int c = min(max(__ldg(cls + b), 0), n_classes - 1);
    if constexpr (IN_REGS) {
      float v[CE_REGS];
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < CE_REGS; ++j) {
        const int i = lane + 32 * j;
        v[j] = i < n_classes ? z[i] : -INFINITY;
        mx = fmaxf(mx, v[j]);
      }
      mx = warp_max(mx);
      float se = 0.f;
#pragma unroll
      for (int j = 0; j < CE_REGS; ++j)
        if (lane + 32 * j < n_classes) se += expf(v[j] - mx);
      se = warp_sum(se);
      const float inv_se = 1.0f / se;
      float zc = 0.f;
#pragma unroll
      for (int j = 0; j < CE_REGS; ++j) {
        const int i = lane + 32 * j;
        if (i < n_classes) {
          float g = (expf(v[j] - mx) * inv_se - (i == c ? 1.f : 0.f)) * inv_b;
          if (relu_mask && !(v[j] > 0.f)) g = 0.f;
          g = apply_round(g, dz_round);
          if constexpr (sizeof(TDz) == 2) dz[(int64_t)b * ld_dz + i] = __float2bfloat16_rn(g);
          else dz[(int64_t)b * ld_dz + i] = g;
          if (i == c) zc = v[j];
        }
      }
      zc = warp_sum(zc);                       // exactly one lane holds the class's logit, the others 0
      if (lane == 0) acc += logf(se) - (zc - mx);
    } else {
      float mx = -INFINITY;
      for (int i = lane; i < n_classes; i += 32) mx = fmaxf(mx, z[i]);
      mx = warp_max(mx);
      float se = 0.f;
      for (int i = lane; i < n_classes; i += 32) se += expf(z[i] - mx);
      se = warp_sum(se);
      const float inv_se = 1.0f / se;
      for (int i = lane; i < n_classes; i += 32) {
        const float zi = z[i];
        float g = (expf(zi - mx) * inv_se - (i == c ? 1.f : 0.f)) * inv_b;
        if (relu_mask && !(zi > 0.f)) g = 0.f;
        g = apply_round(g, dz_round);
        if constexpr (sizeof(TDz) == 2) dz[(int64_t)b * ld_dz + i] = __float2bfloat16_rn(g);
        else dz[(int64_t)b * ld_dz + i] = g;
      }
      if (lane == 0) acc += logf(se) - (z[c] - mx);
    }
  }
  const float bt = block_sum(acc, red);
  finish_loss(bt, partials, counter, loss_out, loss_dst, inv_b, red);
}

// The update of one layer in one launch.  Parameters, gradients and optimizer state share one flat
// layout [W | b]:
//   blocks [0, bias_blocks): each forms the bias gradient of 8 or 32 columns, db[n] = sum_b dZ[b][n]
//     (32 or 8 row lanes per column, then the lanes in index order: one fixed order, bit-reproducible),
//     stores it and applies the optimizer to those bias elements;
//   the other blocks stream over the weight range, whose gradient the weight-gradient product wrote.
// Both parts refresh the reduced-precision operand copy.
template <int OPT, int OPDT>
__global__ void __launch_bounds__(256)
update_kernel(UpdateArgs u, int bias_blocks, int bias_cols) {
  pdl_wait();
  pdl_trigger();
  float inv_bc1 = 1.0f, inv_bc2 = 1.0f;
  if constexpr (OPT == SEG_ADAM) { inv_bc1 = 1.0f / __ldg(u.bc); inv_bc2 = 1.0f / __ldg(u.bc + 1); }
  if ((int)blockIdx.x < bias_blocks) {
    // small batches: 8 columns x 32 row lanes per block, so that the walk over the batch is only batch / 32
    // loads deep and these blocks finish inside the streaming part even when the layer is small;
    // large batches: 32 columns x 8 row lanes (whole 64- or 128-byte row segments per warp)
    __shared__ float part[32][33];
    const int cols = bias_cols, lanes = 256 / bias_cols;
    const int c = threadIdx.x % cols, rl = threadIdx.x / cols;
    const int col = blockIdx.x * cols + c;
    float acc = 0.f;
    if (col < u.n_bias) {
      if (u.dz_dt == DT_BF16) {
        const __nv_bfloat16* dz = reinterpret_cast<const __nv_bfloat16*>(u.dz);
#pragma unroll 8
        for (int b = rl; b < u.batch; b += lanes) acc += __bfloat162float(dz[(int64_t)b * u.ld_dz + col]);
      } else {
        const float* dz = reinterpret_cast<const float*>(u.dz);
#pragma unroll 8
        for (int b = rl; b < u.batch; b += lanes) acc += dz[(int64_t)b * u.ld_dz + col];
      }
    }
    part[rl][c] = acc;
    __syncthreads();
    if (rl == 0 && col < u.n_bias) {
      float g = 0.f;
      for (int r = 0; r < lanes; ++r) g += part[r][c];
      const int64_t i = u.bias_off + col;
      u.g_bias[col] = g;
      float p = u.p[i], m = 0.f, v = 0.f;
      if constexpr (OPT != SEG_SGD) m = u.s1[i];
      if constexpr (OPT == SEG_ADAM) v = u.s2[i];
      opt_step<OPT>(p, g, m, v, u, inv_bc1, inv_bc2);
      if constexpr (OPT != SEG_SGD) u.s1[i] = m;
      if constexpr (OPT == SEG_ADAM) u.s2[i] = v;
      u.p[i] = p;
      if constexpr (OPDT == DT_BF16) {
        reinterpret_cast<__nv_bfloat16*>(u.p_op)[i] = __float2bfloat16_rn(p);
      } else {
        if (u.p_op != nullptr) reinterpret_cast<float*>(u.p_op)[i] = apply_round(p, u.op_round);
      }
    }
    return;
  }
  const int64_t n4 = u.n >> 2;
  float4* __restrict__ p4 = reinterpret_cast<float4*>(u.p);
  const float4* __restrict__ g4 = reinterpret_cast<const float4*>(u.g);
  float4* __restrict__ s14 = reinterpret_cast<float4*>(u.s1);
  float4* __restrict__ s24 = reinterpret_cast<float4*>(u.s2);
  const int64_t stride = (int64_t)(gridDim.x - bias_blocks) * blockDim.x;
  for (int64_t i = (int64_t)(blockIdx.x - bias_blocks) * blockDim.x + threadIdx.x; i < n4; i += stride) {
    const float4 p = p4[i];
    const float4 g = g4[i];
    float pv[4] = {p.x, p.y, p.z, p.w};
    const float gv[4] = {g.x, g.y, g.z, g.w};
    float mv[4] = {0.f, 0.f, 0.f, 0.f}, vv[4] = {0.f, 0.f, 0.f, 0.f};
    if constexpr (OPT != SEG_SGD) { const float4 m = s14[i]; mv[0] = m.x; mv[1] = m.y; mv[2] = m.z; mv[3] = m.w; }
    if constexpr (OPT == SEG_ADAM) { const float4 v = s24[i]; vv[0] = v.x; vv[1] = v.y; vv[2] = v.z; vv[3] = v.w; }
#pragma unroll
    for (int k = 0; k < 4; ++k) opt_step<OPT>(pv[k], gv[k], mv[k], vv[k], u, inv_bc1, inv_bc2);
    if constexpr (OPT != SEG_SGD) s14[i] = make_float4(mv[0], mv[1], mv[2], mv[3]);
    if constexpr (OPT == SEG_ADAM) s24[i] = make_float4(vv[0], vv[1], vv[2], vv[3]);
    p4[i] = make_float4(pv[0], pv[1], pv[2], pv[3]);
    if constexpr (OPDT == DT_BF16) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(pv[0], pv[1]);
      __nv_bfloat162 hi = __floats2bfloat162_rn(pv[2], pv[3]);
      uint2 packed;
      packed.x = *reinterpret_cast<uint32_t*>(&lo);
      packed.y = *reinterpret_cast<uint32_t*>(&hi);
      reinterpret_cast<uint2*>(u.p_op)[i] = packed;
    } else if constexpr (OPDT == DT_F32) {
      if (u.p_op != nullptr) {
        reinterpret_cast<float4*>(u.p_op)[i] =
            make_float4(apply_round(pv[0], u.op_round), apply_round(pv[1], u.op_round),
                        apply_round(pv[2], u.op_round), apply_round(pv[3], u.op_round));
      }
    }
  }
}

__global__ void __launch_bounds__(256)
copy2d_kernel(void* dst, int dst_dt, int64_t ld_dst, const void* src, int src_dt, int64_t ld_src,
              int64_t rows, int64_t cols, int round) {
  pdl_wait();
  pdl_trigger();
  const int64_t total = rows * cols;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total;
       e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = e / cols, c = e % cols;
    const float v = apply_round(load_as_float(src, src_dt, r * ld_src + c), round);
    store_from_float(dst, dst_dt, r * ld_dst + c, v);
  }
}

__global__ void __launch_bounds__(256)
stage_inputs_kernel(void* dst, int dt, int64_t ld_dst, const void* src, int64_t ld_src, int rows, int cols,
                    int round, int32_t* cls_dst, const int32_t* cls_src, unsigned long long* t, float* bc,
                    float beta1, float beta2, const float* gather_src, float* loss_out, float** loss_dst,
                    int n_classes, int* dev_status) {
  pdl_wait();
  pdl_trigger();
  const int64_t total = (int64_t)rows * cols;
  // The last block only keeps the books (the two double-precision powers take longer than a copying thread's
  // share of a small batch; in a block of their own they run beside the copy instead of in front of it).
  const int copy_blocks = (int)gridDim.x - 1;
  if ((int)blockIdx.x == copy_blocks) {
    if (threadIdx.x == 0) {
      if (loss_dst != nullptr) *loss_dst = loss_out;   // where this step's loss kernel writes the loss
      if (t != nullptr) {                              // step counter and Adam bias corrections of this step
        const unsigned long long step = *t + 1ull;
        *t = step;
        bc[0] = (float)(1.0 - pow((double)beta1, (double)step));
        bc[1] = (float)(1.0 - pow((double)beta2, (double)step));
      }
    }
    return;
  }
  const int64_t tid = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  const int64_t n_threads = (int64_t)copy_blocks * blockDim.x;
  const int esz = dt == DT_BF16 ? 2 : 4;
  const bool dst_wide = ((cols * esz) & 15) == 0 && ((ld_dst * esz) & 15) == 0 &&
                        (reinterpret_cast<uintptr_t>(dst) & 15u) == 0;
  if (gather_src != nullptr && dst_wide && (cols & 7) == 0) {
    // the input of sample r is row cls[r] of an fp32 label matrix (the fully separate variant): eight
    // columns per thread and pass, 16-byte loads of the label row, one or two 16-byte stores
    const int groups_per_row = cols / 8;
    const int64_t n_groups = (int64_t)rows * groups_per_row;
    for (int64_t v = tid; v < n_groups; v += n_threads) {
      const int r = (int)(v / groups_per_row), c = (int)(v - (int64_t)r * groups_per_row) * 8;
      const int k = min(max(__ldg(cls_src + r), 0), n_classes - 1);
      const float4 q0 = __ldg(reinterpret_cast<const float4*>(gather_src + (int64_t)k * cols + c));
      const float4 q1 = __ldg(reinterpret_cast<const float4*>(gather_src + (int64_t)k * cols + c + 4));
      float f[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
      if (dt == DT_BF16) {
        __nv_bfloat162 p0 = __floats2bfloat162_rn(f[0], f[1]), p1 = __floats2bfloat162_rn(f[2], f[3]);
        __nv_bfloat162 p2 = __floats2bfloat162_rn(f[4], f[5]), p3 = __floats2bfloat162_rn(f[6], f[7]);
        uint4 q;
        q.x = *reinterpret_cast<uint32_t*>(&p0); q.y = *reinterpret_cast<uint32_t*>(&p1);
        q.z = *reinterpret_cast<uint32_t*>(&p2); q.w = *reinterpret_cast<uint32_t*>(&p3);
        *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(dst) + (int64_t)r * ld_dst + c) = q;
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) f[j] = apply_round(f[j], round);
        float* drow = reinterpret_cast<float*>(dst) + (int64_t)r * ld_dst + c;
        *reinterpret_cast<float4*>(drow) = make_float4(f[0], f[1], f[2], f[3]);
        *reinterpret_cast<float4*>(drow + 4) = make_float4(f[4], f[5], f[6], f[7]);
      }
    }
  } else if (gather_src == nullptr && dst_wide && ((ld_src * esz) & 15) == 0 &&
             (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
    // 16 bytes per access: rows are whole numbers of 16-byte groups on both sides
    const int vec_per_row = cols * esz / 16;
    const int64_t n_vec = (int64_t)rows * vec_per_row;
    const char* sb = reinterpret_cast<const char*>(src);
    char* db = reinterpret_cast<char*>(dst);
    for (int64_t v = tid; v < n_vec; v += n_threads) {
      const int64_t r = v / vec_per_row, c = v % vec_per_row;
      uint4 q = __ldg(reinterpret_cast<const uint4*>(sb + r * ld_src * esz) + c);
      if (round == RND_TF32 && dt == DT_F32) {
        q.x = __float_as_uint(round_tf32_rne(__uint_as_float(q.x)));
        q.y = __float_as_uint(round_tf32_rne(__uint_as_float(q.y)));
        q.z = __float_as_uint(round_tf32_rne(__uint_as_float(q.z)));
        q.w = __float_as_uint(round_tf32_rne(__uint_as_float(q.w)));
      }
      reinterpret_cast<uint4*>(db + r * ld_dst * esz)[c] = q;
    }
  } else {
    for (int64_t e = tid; e < total; e += n_threads) {
      const int64_t r = e / cols, c = e % cols;
      float raw;
      if (gather_src) {
        const int k = min(max(__ldg(cls_src + r), 0), n_classes - 1);
        raw = __ldg(gather_src + (int64_t)k * cols + c);
      } else {
        raw = load_as_float(src, dt, r * ld_src + c);
      }
      store_from_float(dst, dt, r * ld_dst + c, apply_round(raw, round));
    }
  }
  // class indices: clamped into [0, n_classes); one outside that range is recorded in the status word
  for (int64_t i = tid; i < rows; i += n_threads) {
    const int k = cls_src[i];
    const int kc = min(max(k, 0), n_classes - 1);
    if (kc != k && dev_status != nullptr) atomicOr(dev_status, (int)DEV_BAD_CLASS);
    cls_dst[i] = kc;
  }
}

int grid_for(int64_t work_items, int threads, int max_blocks) {
  int64_t b = (work_items + threads - 1) / threads;
  if (b < 1) b = 1;
  return (int)(b < max_blocks ? b : max_blocks);
}

}  // namespace

int loss_max_partials() { return kMaxLossBlocks; }

// Eight columns per thread when every row segment involved is 16-byte aligned, one otherwise.
bool mse_wide(const void* out, int64_t ld_out, const void* dz, int64_t ld_dz, const float* sil, int n_p) {
  return (n_p & 7) == 0 && (ld_out & 7) == 0 && (ld_dz & 7) == 0 &&
         ((reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(dz) | reinterpret_cast<uintptr_t>(sil)) & 15u) == 0;
}

cudaError_t launch_mse_loss(const void* out, int out_dt, int64_t ld_out, const int32_t* cls,
                            const float* sil, int n_classes, int n_p, int batch, int relu_mask, void* dz,
                            int dz_dt, int dz_round, int64_t ld_dz, float* partials,
                            unsigned int* counter, float* const* loss_dst, cudaStream_t s) {
  float* const loss_out = nullptr;
  const bool wide = mse_wide(out, ld_out, dz, ld_dz, sil, n_p);
  const int grid = grid_for((int64_t)batch * n_p, kLossThreads * (wide ? 16 : 4), kMaxLossBlocks);
#define SEGK_MSE(TO, TD, V)                                                                              \
  launch_k(mse_loss_kernel<TO, TD, V>, dim3(grid), dim3(kLossThreads), 0, s, (const TO*)out, ld_out, cls, \
           sil, n_classes, n_p, batch, relu_mask, (TD*)dz, dz_round, ld_dz, partials, counter, loss_out, loss_dst)
  if (out_dt == DT_BF16 && dz_dt == DT_BF16) {
    if (wide) SEGK_MSE(__nv_bfloat16, __nv_bfloat16, 8); else SEGK_MSE(__nv_bfloat16, __nv_bfloat16, 1);
  } else if (out_dt == DT_F32 && dz_dt == DT_F32) {
    if (wide) SEGK_MSE(float, float, 8); else SEGK_MSE(float, float, 1);
  } else {
    return cudaErrorInvalidValue;
  }
#undef SEGK_MSE
  return cudaGetLastError();
}

cudaError_t launch_softmax_ce_loss(const float* logits, int64_t ld_logits, const int32_t* cls,
                                   int n_classes, int batch, int relu_mask, void* dz, int dz_dt,
                                   int dz_round, int64_t ld_dz, float* partials,
                                   unsigned int* counter, float* const* loss_dst, cudaStream_t s) {
  float* const loss_out = nullptr;
  const int warps = kLossThreads / 32;
  const int grid = grid_for(batch, warps, kMaxLossBlocks);
  const bool in_regs = n_classes <= 32 * CE_REGS;
#define SEGK_CE(TD, R)                                                                                         \
  launch_k(softmax_ce_kernel<TD, R>, dim3(grid), dim3(kLossThreads), 0, s, logits, ld_logits, cls, n_classes, \
           batch, relu_mask, (TD*)dz, dz_round, ld_dz, partials, counter, loss_out, loss_dst)
  if (dz_dt == DT_BF16) {
    if (in_regs) SEGK_CE(__nv_bfloat16, true); else SEGK_CE(__nv_bfloat16, false);
  } else {
    if (in_regs) SEGK_CE(float, true); else SEGK_CE(float, false);
  }
#undef SEGK_CE
  return cudaGetLastError();
}

cudaError_t launch_update(const UpdateArgs& u, cudaStream_t s) {
  if (u.n & 3) return cudaErrorInvalidValue;
  const int bias_cols = (u.batch <= 1024 || u.n_bias <= 256) ? 8 : 32;   // narrow layers: few blocks either way, keep the walk short
  const int bias_blocks = (u.dz != nullptr && u.n_bias > 0) ? (u.n_bias + bias_cols - 1) / bias_cols : 0;
  if (u.n == 0 && bias_blocks == 0) return cudaSuccess;
  // two rounds of resident blocks (8 per SM): measured 5.6 TB/s against 4.9 with one round on the 67 M-element
  // momentum update, no difference for Adam; streaming (evict-first) loads and stores measured no better
  const int grid = bias_blocks + (u.n > 0 ? grid_for(u.n >> 2, 256, 148 * 16) : 0);
  const bool bf = (u.p_op != nullptr && u.op_dt == DT_BF16);
#define SEGK_UPD(OPT)                                                      \
  if (bf) launch_k(update_kernel<OPT, DT_BF16>, dim3(grid), dim3(256), 0, s, u, bias_blocks, bias_cols);             \
  else launch_k(update_kernel<OPT, DT_F32>, dim3(grid), dim3(256), 0, s, u, bias_blocks, bias_cols)
  switch (u.optimizer) {
    case SEG_SGD: SEGK_UPD(SEG_SGD); break;
    case SEG_SGD_MOMENTUM: SEGK_UPD(SEG_SGD_MOMENTUM); break;
    case SEG_ADAM: SEGK_UPD(SEG_ADAM); break;
    default: return cudaErrorInvalidValue;
  }
#undef SEGK_UPD
  return cudaGetLastError();
}

cudaError_t launch_stage_inputs(void* dst, int dt, int64_t ld_dst, const void* src, int64_t ld_src, int rows,
                                int cols, int round, int32_t* cls_dst, const int32_t* cls_src,
                                unsigned long long* t, float* bc, float beta1, float beta2,
                                const float* gather_src, float* loss_out, float** loss_dst,
                                int n_classes, int* dev_status, cudaStream_t s) {
  const int esz = dt == DT_BF16 ? 2 : 4;
  const int grid = grid_for((int64_t)rows * cols * esz / 16, 256, 148 * 8) + 1;   // one 16-byte group per thread and pass; + the bookkeeping block
  launch_k(stage_inputs_kernel, dim3(grid), dim3(256), 0, s, dst, dt, ld_dst, src, ld_src, rows, cols, round, cls_dst, cls_src, t, bc,
                                           beta1, beta2, gather_src, loss_out, loss_dst, n_classes, dev_status);
  return cudaGetLastError();
}

cudaError_t launch_copy2d(void* dst, int dst_dt, int64_t ld_dst, const void* src, int src_dt,
                          int64_t ld_src, int64_t rows, int64_t cols, int round, cudaStream_t s) {
  if (rows <= 0 || cols <= 0) return cudaSuccess;
  const int grid = grid_for(rows * cols, 256 * 4, 148 * 8);
  launch_k(copy2d_kernel, dim3(grid), dim3(256), 0, s, dst, dst_dt, ld_dst, src, src_dt, ld_src, rows, cols, round);
  return cudaGetLastError();
}

}  // namespace segk

// ---- entry point that allocates nothing ---------------------------------------------------------
// The intermediate-label loss for callers that may not allocate device memory: plug-ins that run
// inside another program's fixed memory budget, latency-bound loops that cannot afford the device
// synchronisation cudaMalloc implies, code that is handed a stream and buffers but no allocator.
// The reduction scratch the loss kernel needs (one partial sum per thread block and the arrival
// counter) lives in the file-scope device array below instead of a handle's workspace.  The array
// exists once on every device that loads this library and is held until the process exits.
namespace segk {
namespace {

constexpr size_t kStaticScratchBytes = 8192;           // 1024 block partials (4 KiB) + arrival counter
static __device__ __align__(256) unsigned char g_static_loss_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_static_scratch_ptr[kMaxDevices] = {};          // device address of the array, per device

// In host code the array's name is only a handle for the runtime, not a device address; the
// address a kernel can use comes from cudaGetSymbolAddress, asked once per device with that
// device current.
cudaError_t static_scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (g_static_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_loss_scratch);
    if (e != cudaSuccess) return e;
    g_static_scratch_ptr[dev] = p;
  }
  *out = g_static_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace segk

extern "C" SEG_API seg_status seg_label_loss_noalloc(const float* out, const int32_t* cls, const float* sil,
                                                     int32_t n_classes, int32_t n_p, int32_t batch,
                                                     int32_t relu_mask, float* dz, float* loss_out,
                                                     void* stream) {
  using namespace segk;
  if (!out || !cls || !sil || !dz) return SEG_ERR_INVALID_ARG;
  if (n_classes < 1 || n_p < 1 || batch < 1) return SEG_ERR_SHAPE;
  if (n_p > SEG_NOALLOC_MAX_WIDTH || batch > SEG_NOALLOC_MAX_BATCH) return SEG_ERR_SHAPE;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  void* scratch = nullptr;
  if (static_scratch_address(&scratch) != cudaSuccess) { cudaGetLastError(); return SEG_ERR_CUDA; }
  float* partials = reinterpret_cast<float*>(scratch);
  unsigned int* counter = reinterpret_cast<unsigned int*>(reinterpret_cast<unsigned char*>(scratch) + 4096);
  // the array keeps whatever the previous call left: the arrival counter must start at zero
  if (cudaMemsetAsync(counter, 0, sizeof(unsigned int), s) != cudaSuccess) { cudaGetLastError(); return SEG_ERR_CUDA; }
  const bool wide = mse_wide(out, n_p, dz, n_p, sil, n_p);
  const int grid = grid_for((int64_t)batch * n_p, kLossThreads * (wide ? 16 : 4), kMaxLossBlocks);
  if (wide)
    mse_loss_kernel<float, float, 8><<<grid, kLossThreads, 0, s>>>(out, n_p, cls, sil, n_classes, n_p, batch, relu_mask ? 1 : 0,
                                                                  dz, RND_NONE, n_p, partials, counter, loss_out, nullptr);
  else
    mse_loss_kernel<float, float, 1><<<grid, kLossThreads, 0, s>>>(out, n_p, cls, sil, n_classes, n_p, batch, relu_mask ? 1 : 0,
                                                                  dz, RND_NONE, n_p, partials, counter, loss_out, nullptr);
  if (cudaGetLastError() != cudaSuccess) return SEG_ERR_CUDA;
  return SEG_OK;
}
