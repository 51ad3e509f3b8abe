// The whole training step of a small fp32 segment in two launches (Section 2: forward through the
// segment's layers, loss against the intermediate labels of the samples' classes or, in the final
// segment, against the class labels, backward, update; Section 3: layers of 80, 60 and 47 units).
//
// A segment whose layers are at most kSmallMaxWidth wide runs ten or more dependent launches of a few
// microseconds each when every product, the loss and every update is a kernel of its own.  Here
//   1. small_fwd_bwd_kernel gives every CTA a slice of R rows of the batch and carries it through the
//      whole chain: input staging (class clamp, gather of label rows), all forward products with bias
//      and ReLU, the loss and dZ of the last layer, and the dgrad chain.  Activations and dZ of the slice
//      stay in shared memory (stored k-major, so that a thread reads its rows with 16-byte loads); the
//      weights of all products of the chain arrive as one stream of 64-row tiles through a cp.async ring.
//      Every activation and dZ also goes to global memory, where the second kernel (and
//      seg_get_activation) reads it.
//   2. small_wgrad_update_kernel forms dW_l = dZ_l^T A_{l-1} of all layers in one grid of 64 x 64 tiles,
//      the batch split over several CTAs per tile; the bias gradient is the column a ones-vector appended
//      to A_{l-1} yields.  The last CTA of a tile to arrive adds the partial tiles in split order (a fixed
//      order: bit-reproducible), stores the gradient and applies the optimizer to its elements.
#include <algorithm>
#include <atomic>

#include "common.cuh"

namespace segk {
namespace {

constexpr int SS_THREADS = 256;
constexpr int SS_KT = 64;                                   // contraction rows per staged weight tile
constexpr int SS_STAGES = 3;                                // weight tiles in flight (cp.async groups)
constexpr int SS_KF_LD = SS_KT + 4;                         // k-fast tile [128 n][68]: a lane reads 4 k with one conflict-free 16-byte load
constexpr int SS_NF_LD = kSmallMaxWidth + 4;                // n-fast tile [64 k][132]
constexpr int SS_STAGE_FLOATS = kSmallMaxWidth * SS_KF_LD;  // the larger of the two layouts
constexpr int SS_CHUNKS = kSmallMaxWidth * SS_KT / 4 / SS_THREADS;   // 16-byte chunks of a tile per thread
static_assert(SS_STAGE_FLOATS >= SS_KT * SS_NF_LD, "stage size");
static_assert(kSmallMaxWidth == 128 && SS_THREADS == 256 && SS_KT == 64, "thread mappings below");

__device__ __forceinline__ void cp_async16(float* smem_dst, const float* src, bool valid) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  const int bytes = valid ? 16 : 0;                         // 0: nothing is read, the 16 bytes are zero-filled
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// One matrix product of the chain, seen from the weight side: out[r][n] = sum_k left[k][r] * Wmat(k, n) with
// Wmat(k, n) = W[n * ldw + k] (k_fast: a forward product, A W^T) or W[k * ldw + n] (dgrad, dZ W).
struct Phase { const float* W; int ldw, K, N; bool k_fast; };

__device__ __forceinline__ Phase phase_of(const SmallStep& p, int ph) {
  Phase q;
  const int L = p.n_layers;
  const int l = ph < L ? ph : 2 * L - 1 - ph;               // forward 0 .. L-1, then dgrad L-1 .. 1
  q.k_fast = ph < L;
  q.W = p.params + p.w_off[l]; q.ldw = (int)p.ldw[l];
  q.K = q.k_fast ? p.widths[l] : p.widths[l + 1];
  q.N = q.k_fast ? p.widths[l + 1] : p.widths[l];
  return q;
}

// The stream of weight tiles of the whole chain (all forward products, then the dgrad chain): the weights depend
// on nothing the kernel computes, so the tiles of a later product are in flight while an earlier one finishes.
// A tile is rows k0 .. k0+63 of Wmat, copied asynchronously, 8 chunks of 16 bytes per thread.  Rows of W are 16-byte
// aligned and their pitch is a multiple of 8 floats, so a chunk never crosses a row's allocation; what it carries
// beyond K or N is never read by the arithmetic.  Per phase every thread keeps the source and destination of its
// first chunk; the others follow at fixed strides (k-fast: thread -> 4 k of row n = tid / 16 + 16 i; n-fast:
// 4 n of row k = tid / 32 + 8 i).
struct TileStream {
  const SmallStep& p;
  float* stages;
  int n_phases, ph = 0, k0 = 0, stage = 0;
  Phase q;
  const float* src = nullptr;
  int c4 = 0, r0 = 0, r_step = 0, dst = 0, dst_step = 0, src_step = 0;
  __device__ TileStream(const SmallStep& pp, float* st) : p(pp), stages(st), n_phases(2 * pp.n_layers - 1) { load_phase(); }
  __device__ __forceinline__ void load_phase() {
    q = phase_of(p, ph);
    const int tid = threadIdx.x;
    if (q.k_fast) { c4 = 4 * (tid & 15); r0 = tid >> 4; r_step = 16; dst = r0 * SS_KF_LD + c4; dst_step = 16 * SS_KF_LD; }
    else { c4 = 4 * (tid & 31); r0 = tid >> 5; r_step = 8; dst = r0 * SS_NF_LD + c4; dst_step = 8 * SS_NF_LD; }
    src = q.W + (int64_t)r0 * q.ldw + c4;
    src_step = r_step * q.ldw;
  }
  __device__ __forceinline__ void issue_next() {           // always commits a group, so that the group count is uniform
    if (ph < n_phases) {
      float* d = stages + stage * SS_STAGE_FLOATS + dst;
      if (q.k_fast) {
        const bool col_ok = k0 + c4 < q.ldw;
        const float* s0 = src + k0;
#pragma unroll
        for (int i = 0; i < SS_CHUNKS; ++i) {
          const bool ok = col_ok && r0 + r_step * i < q.N;
          cp_async16(d + i * dst_step, ok ? s0 + i * src_step : q.W, ok);
        }
      } else {
        const bool col_ok = c4 < q.ldw;
        const float* s0 = src + (int64_t)k0 * q.ldw;
#pragma unroll
        for (int i = 0; i < SS_CHUNKS; ++i) {
          const bool ok = col_ok && k0 + r0 + r_step * i < q.K;
          cp_async16(d + i * dst_step, ok ? s0 + i * src_step : q.W, ok);
        }
      }
      k0 += SS_KT;
      if (k0 >= q.K) {
        ++ph; k0 = 0;
        if (ph < n_phases) load_phase();
      }
    }
    cp_async_commit();
    stage = stage + 1 == SS_STAGES ? 0 : stage + 1;
  }
};

// acc[j] += sum_k left[k][rg * RPT + j] * Wmat(k, n) for this thread's column n and its RPT rows; left is the
// slice's left operand in shared memory, k-major with R rows per k.  All threads of the CTA call it; `cstage` is the
// stage the next tile to consume sits in.
template <int R, int RPT>
__device__ __forceinline__ void rows_times_weights(float (&acc)[RPT], const float* left, const Phase& q, TileStream& ts,
                                                   int& cstage, int rg, int n) {
  for (int k0 = 0; k0 < q.K; k0 += SS_KT) {
    cp_async_wait<SS_STAGES - 2>();      // this tile's group has landed (for this thread's copies) ...
    __syncthreads();                     // ... and for everyone's; all threads are done with the previous tile
    ts.issue_next();                     // refills the stage the previous tile occupied
    const float* stage = ts.stages + cstage * SS_STAGE_FLOATS;
    cstage = cstage + 1 == SS_STAGES ? 0 : cstage + 1;
    const int kmax = min(SS_KT, q.K - k0);
    if (n < q.N) {
      const float* ap = left + (size_t)k0 * R + rg * RPT;
      auto fma_row = [&](int kk, float w) {
#pragma unroll
        for (int u = 0; u < RPT / 4; ++u) {
          const float4 a = *reinterpret_cast<const float4*>(ap + kk * R + 4 * u);
          acc[4 * u + 0] = fmaf(a.x, w, acc[4 * u + 0]);
          acc[4 * u + 1] = fmaf(a.y, w, acc[4 * u + 1]);
          acc[4 * u + 2] = fmaf(a.z, w, acc[4 * u + 2]);
          acc[4 * u + 3] = fmaf(a.w, w, acc[4 * u + 3]);
        }
      };
      if (q.k_fast) {
        const float* ws = stage + n * SS_KF_LD;
        int kk = 0;
#pragma unroll 4
        for (; kk + 4 <= kmax; kk += 4) {
          const float4 w = *reinterpret_cast<const float4*>(ws + kk);
          fma_row(kk, w.x); fma_row(kk + 1, w.y); fma_row(kk + 2, w.z); fma_row(kk + 3, w.w);
        }
        for (; kk < kmax; ++kk) fma_row(kk, ws[kk]);
      } else {
#pragma unroll 4
        for (int kk = 0; kk < kmax; ++kk) fma_row(kk, stage[kk * SS_NF_LD + n]);
      }
    }
  }
}

// Shared-memory floats of small_fwd_bwd_kernel: weight stages, two dZ buffers, one activation buffer per layer boundary.
size_t fwd_bwd_smem_floats(const SmallStep& p, int R) {
  size_t f = (size_t)SS_STAGES * SS_STAGE_FLOATS + 2 * (size_t)kSmallMaxWidth * R;
  for (int l = 0; l <= p.n_layers; ++l) f += (size_t)p.widths[l] * R;
  return f;
}

template <int R>
__global__ void __launch_bounds__(SS_THREADS)
small_fwd_bwd_kernel(const __grid_constant__ SmallStep p, const float* __restrict__ x, const int32_t* __restrict__ cls,
                     const float* __restrict__ gather, float* loss_to) {
  constexpr int RPT = R / 2;
  extern __shared__ __align__(16) float ss_smem[];
  __shared__ int cls_s[R];
  __shared__ float red[32];
  pdl_wait();
  pdl_trigger();
  const int tid = threadIdx.x, n = tid & (kSmallMaxWidth - 1), rg = tid >> 7;
  const int L = p.n_layers;
  const int row0 = blockIdx.x * R;
  const int nv = min(R, p.batch - row0);
  float* dzT[2] = {ss_smem + SS_STAGES * SS_STAGE_FLOATS, ss_smem + SS_STAGES * SS_STAGE_FLOATS + kSmallMaxWidth * R};
  float* aT0 = dzT[1] + kSmallMaxWidth * R;
  auto aT = [&](int l) {               // activation of layer boundary l (0: the segment's input), [widths[l]][R]
    float* q = aT0;
    for (int i = 0; i < l; ++i) q += p.widths[i] * R;
    return q;
  };
  TileStream ts(p, ss_smem);
  int cstage = 0;
#pragma unroll
  for (int i = 0; i < SS_STAGES - 1; ++i) ts.issue_next();

  // step counter, Adam's bias corrections, where the loss goes; class indices of the slice (clamped)
  if (blockIdx.x == 0 && tid == 0) {
    const unsigned long long step = *p.t + 1ull;
    *p.t = step;
    if (p.optimizer == SEG_ADAM) {      // the only reader of the bias corrections; two double-precision powers cost over a microsecond
      p.bc[0] = (float)(1.0 - pow((double)p.beta1, (double)step));
      p.bc[1] = (float)(1.0 - pow((double)p.beta2, (double)step));
    }
    *p.loss_dst = loss_to;
  }
  if (tid < R) {
    int c = 0;
    if (tid < nv) {
      c = cls[row0 + tid];
      if (c < 0 || c >= p.n_classes) {
        atomicOr(p.dev_status, (int)DEV_BAD_CLASS);
        c = min(max(c, 0), p.n_classes - 1);
      }
      p.cls_stage[row0 + tid] = c;
    }
    cls_s[tid] = c;
  }
  __syncthreads();

  // the slice's input rows: the caller's batch, or the previous cut's label rows gathered by class
  {
    const int n0 = p.widths[0];
    for (int k = tid; k < n0; k += SS_THREADS) {
      float v[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        v[r] = 0.f;
        if (r < nv) {
          const float* src = gather ? gather + (int64_t)cls_s[r] * n0 : x + (int64_t)(row0 + r) * n0;
          v[r] = src[k];
        }
      }
#pragma unroll
      for (int r = 0; r < R; ++r)
        if (r < nv) p.act[0][(int64_t)(row0 + r) * p.ld_act[0] + k] = v[r];
#pragma unroll
      for (int u = 0; u < R / 4; ++u)
        *reinterpret_cast<float4*>(aT0 + (size_t)k * R + 4 * u) = make_float4(v[4 * u], v[4 * u + 1], v[4 * u + 2], v[4 * u + 3]);
    }
  }

  // forward:  A_l = act(A_{l-1} W_l^T + b_l)   (the first wait of every product orders the shared-memory
  // writes of the step before it)
  for (int l = 0; l < L; ++l) {
    const Phase q = phase_of(p, l);
    float acc[RPT];
#pragma unroll
    for (int j = 0; j < RPT; ++j) acc[j] = 0.f;
    const float b = n < q.N ? p.params[p.b_off[l] + n] : 0.f;      // in flight during the product
    rows_times_weights<R, RPT>(acc, aT(l), q, ts, cstage, rg, n);
    if (n < q.N) {
      const bool relu = (l < L - 1) || p.last_relu;
      float* an = aT(l + 1) + (size_t)n * R + rg * RPT;
#pragma unroll
      for (int j = 0; j < RPT; ++j) {
        float v = acc[j] + b;
        if (relu) v = fmaxf(v, 0.f);
        an[j] = v;
        const int r = rg * RPT + j;
        if (r < nv) p.act[l + 1][(int64_t)(row0 + r) * p.ld_act[l + 1] + n] = v;
      }
    }
  }
  __syncthreads();

  // loss and dZ of the last layer
  const int NL = p.widths[L];
  const float* zT = aT(L);
  float* dz_cur = dzT[0];
  float* dz_g = p.dz[L - 1];
  const int64_t ld_dzL = p.ld_act[L];
  float lsum = 0.f;
  if (!p.is_final) {
    // mean squared error against the label row of the sample's class:  dZ = 2 (a - t) / (B N_P) * [a > 0]
    const float gscale = 2.0f / (float)((int64_t)p.batch * NL);
    if (n < NL) {
      float tgt[RPT];
#pragma unroll
      for (int j = 0; j < RPT; ++j) tgt[j] = rg * RPT + j < nv ? __ldg(p.sil + (int64_t)cls_s[rg * RPT + j] * NL + n) : 0.f;
#pragma unroll
      for (int j = 0; j < RPT; ++j) {
        const int r = rg * RPT + j;
        float g = 0.f;
        if (r < nv) {
          const float a = zT[(size_t)n * R + r];
          const float d = a - tgt[j];
          lsum = fmaf(d, d, lsum);
          g = d * gscale;
          if (p.last_relu && !(a > 0.f)) g = 0.f;
          dz_g[(int64_t)(row0 + r) * ld_dzL + n] = g;
        }
        dz_cur[(size_t)n * R + r] = g;
      }
    }
  } else {
    // softmax cross-entropy, one warp per row:  dZ = (softmax(z) - onehot) / B
    const int lane = tid & 31, warp = tid >> 5;
    const float inv_b = 1.0f / (float)p.batch;
    for (int r = warp; r < R; r += SS_THREADS / 32) {
      float v[kSmallMaxWidth / 32];
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < kSmallMaxWidth / 32; ++j) {
        const int i = lane + 32 * j;
        v[j] = i < NL ? zT[(size_t)i * R + r] : -INFINITY;
        mx = fmaxf(mx, v[j]);
      }
      mx = warp_max(mx);
      float se = 0.f;
#pragma unroll
      for (int j = 0; j < kSmallMaxWidth / 32; ++j)
        if (lane + 32 * j < NL) se += expf(v[j] - mx);
      se = warp_sum(se);
      const float inv_se = 1.0f / se;
      const int c = cls_s[r];
      float zc = 0.f;
#pragma unroll
      for (int j = 0; j < kSmallMaxWidth / 32; ++j) {
        const int i = lane + 32 * j;
        if (i < NL) {
          float g = 0.f;
          if (r < nv) {
            g = (expf(v[j] - mx) * inv_se - (i == c ? 1.f : 0.f)) * inv_b;
            if (p.last_relu && !(v[j] > 0.f)) g = 0.f;
            dz_g[(int64_t)(row0 + r) * ld_dzL + i] = g;
            if (i == c) zc = v[j];
          }
          dz_cur[(size_t)i * R + r] = g;
        }
      }
      zc = warp_sum(zc);
      if (lane == 0 && r < nv) lsum += logf(se) - (zc - mx);
    }
  }

  // dgrad chain:  dZ_{l-1} = (dZ_l W_l) * [A_{l-1} > 0]
  for (int l = L - 1; l >= 1; --l) {
    const Phase q = phase_of(p, 2 * L - 1 - l);
    float acc[RPT];
#pragma unroll
    for (int j = 0; j < RPT; ++j) acc[j] = 0.f;
    rows_times_weights<R, RPT>(acc, dz_cur, q, ts, cstage, rg, n);
    float* dz_next = (dz_cur == dzT[0]) ? dzT[1] : dzT[0];
    if (n < q.N) {
      const float* al = aT(l) + (size_t)n * R + rg * RPT;
#pragma unroll
      for (int j = 0; j < RPT; ++j) {
        const int r = rg * RPT + j;
        float g = acc[j];
        if (!(al[j] > 0.f)) g = 0.f;
        dz_next[(size_t)n * R + r] = g;
        if (r < nv) p.dz[l - 1][(int64_t)(row0 + r) * p.ld_act[l] + n] = g;
      }
    }
    dz_cur = dz_next;
  }
  cp_async_wait<0>();

  const float bt = block_sum(lsum, red);
  const float scale = p.is_final ? 1.0f / (float)p.batch : 1.0f / (float)((int64_t)p.batch * NL);
  finish_loss(bt, p.loss_partials, p.loss_counter, loss_to, nullptr, scale, red);
}

// ---- weight gradients of all layers, bias gradients and the update ---------------------------------
constexpr int WT = 64, WK = 32, WPAD = 4;

__host__ __device__ inline int wgrad_tiles(int in, int out) { return ((out + WT - 1) / WT) * ((in + 1 + WT - 1) / WT); }

template <int OPT>
__global__ void __launch_bounds__(SS_THREADS)
small_wgrad_update_kernel(SmallStep p, int splits, int k_per_split) {
  pdl_wait();
  pdl_trigger();
  __shared__ bool is_last;
  __shared__ __align__(16) float As[WK][WT + WPAD];
  __shared__ __align__(16) float Bs[WK][WT + WPAD];
  const int tile = blockIdx.x / splits, z = blockIdx.x - tile * splits;
  int l = 0, t = tile;
  for (; l < p.n_layers - 1; ++l) {
    const int nt = wgrad_tiles(p.widths[l], p.widths[l + 1]);
    if (t < nt) break;
    t -= nt;
  }
  const int in = p.widths[l], out = p.widths[l + 1];
  const int tiles_n = (in + 1 + WT - 1) / WT;
  const int m0 = (t / tiles_n) * WT, n0 = (t % tiles_n) * WT;
  const float* __restrict__ dz = p.dz[l];            // (m = o, k = b) at dz[b * ld_dz + o]
  const float* __restrict__ ap = p.act[l];           // (k = b, n = i) at ap[b * ld_a + i];  column `in` is all ones
  const int64_t ld_dz = p.ld_act[l + 1], ld_a = p.ld_act[l];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int k_begin = z * k_per_split, k_end = min(p.batch, k_begin + k_per_split);
  // A k-step of each operand is 32 rows of 64 floats = 512 groups of 4: two per thread.  A group inside the
  // buffer's pitch is one 16-byte load (rows are 32-byte aligned; what lies between the width and the pitch is
  // zero, and products with it are never stored); the group of A_{l-1} that holds column `in` (the ones) or
  // crosses the width is put together element by element.
  constexpr int LD = WT * WK / 4 / SS_THREADS;
  float4 ra[LD], rb[LD];
  float acc[4][4] = {};
  auto fetch = [&](int k0) {
#pragma unroll
    for (int i = 0; i < LD; ++i) {
      const int idx = threadIdx.x + SS_THREADS * i;
      const int c = (idx & 15) * 4, k = k0 + (idx >> 4);
      ra[i] = make_float4(0.f, 0.f, 0.f, 0.f); rb[i] = ra[i];
      if (k < k_end) {
        if (m0 + c + 3 < ld_dz) ra[i] = *reinterpret_cast<const float4*>(dz + (int64_t)k * ld_dz + m0 + c);
        if (n0 + c + 3 < in) {
          rb[i] = *reinterpret_cast<const float4*>(ap + (int64_t)k * ld_a + n0 + c);
        } else {
          float t[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int cc = n0 + c + j;
            t[j] = cc < in ? ap[(int64_t)k * ld_a + cc] : (cc == in ? 1.0f : 0.f);
          }
          rb[i] = make_float4(t[0], t[1], t[2], t[3]);
        }
      }
    }
  };
  if (k_begin < k_end) fetch(k_begin);
  for (int k0 = k_begin; k0 < k_end; k0 += WK) {
#pragma unroll
    for (int i = 0; i < LD; ++i) {
      const int idx = threadIdx.x + SS_THREADS * i;
      *reinterpret_cast<float4*>(&As[idx >> 4][(idx & 15) * 4]) = ra[i];
      *reinterpret_cast<float4*>(&Bs[idx >> 4][(idx & 15) * 4]) = rb[i];
    }
    __syncthreads();
    if (k0 + WK < k_end) fetch(k0 + WK);
#pragma unroll
    for (int k = 0; k < WK; ++k) {
      const float4 a = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  if (splits > 1) {
    float* slot = p.wg_scratch + ((size_t)tile * splits + z) * kSimtTileFloats;
#pragma unroll
    for (int i = 0; i < 4; ++i)
      *reinterpret_cast<float4*>(slot + (ty * 4 + i) * WT + tx * 4) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(p.wg_counters + tile, 1u) == (unsigned)splits - 1u);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const float* base = p.wg_scratch + (size_t)tile * splits * kSimtTileFloats;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    // four partial tiles are loaded before any is added (the loads of one round overlap; a round past the last split
    // adds zeros); the order of the additions stays split by split
    auto part = [&](int s, int i) {
      return __ldcg(reinterpret_cast<const float4*>(base + (size_t)s * kSimtTileFloats + (ty * 4 + i) * WT + tx * 4));
    };
    for (int s = 0; s < splits; s += 4) {
      float4 q[4][4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int i = 0; i < 4; ++i) q[u][i] = s + u < splits ? part(s + u, i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          acc[i][0] += q[u][i].x; acc[i][1] += q[u][i].y; acc[i][2] += q[u][i].z; acc[i][3] += q[u][i].w;
        }
    }
    if (threadIdx.x == 0) p.wg_counters[tile] = 0u;
  }
  float inv_bc1 = 1.0f, inv_bc2 = 1.0f;
  if constexpr (OPT == SEG_ADAM) { inv_bc1 = 1.0f / __ldg(p.bc); inv_bc2 = 1.0f / __ldg(p.bc + 1); }
  // this thread's 16 elements (4 rows of 4 consecutive columns): all loads first (they do not depend on one
  // another), then the arithmetic and the stores.  A row segment that lies wholly inside the weight matrix moves
  // with 16-byte accesses (rows of W are 32-byte aligned and the segment starts at a multiple of 4 columns); the
  // ragged segment at the matrix edge, which also carries the bias element, goes element by element.
  int64_t e[4][4];
  bool wide[4];
  float w[4][4], m[4][4], v[4][4];
  const int c0 = n0 + tx * 4;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int o = m0 + ty * 4 + i;
    wide[i] = o < out && c0 + 3 < in;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = c0 + j;
      e[i][j] = (o >= out || c > in) ? -1 : (c < in ? p.w_off[l] + (int64_t)o * p.ldw[l] + c : p.b_off[l] + o);
      w[i][j] = 0.f; m[i][j] = 0.f; v[i][j] = 0.f;
    }
    if (wide[i]) {
      const float4 q = *reinterpret_cast<const float4*>(p.params + e[i][0]);
      w[i][0] = q.x; w[i][1] = q.y; w[i][2] = q.z; w[i][3] = q.w;
      if constexpr (OPT != SEG_SGD) {
        const float4 t = *reinterpret_cast<const float4*>(p.s1 + e[i][0]);
        m[i][0] = t.x; m[i][1] = t.y; m[i][2] = t.z; m[i][3] = t.w;
      }
      if constexpr (OPT == SEG_ADAM) {
        const float4 t = *reinterpret_cast<const float4*>(p.s2 + e[i][0]);
        v[i][0] = t.x; v[i][1] = t.y; v[i][2] = t.z; v[i][3] = t.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (e[i][j] < 0) continue;
        w[i][j] = p.params[e[i][j]];
        if constexpr (OPT != SEG_SGD) m[i][j] = p.s1[e[i][j]];
        if constexpr (OPT == SEG_ADAM) v[i][j] = p.s2[e[i][j]];
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (e[i][j] >= 0) opt_step<OPT>(w[i][j], acc[i][j], m[i][j], v[i][j], p, inv_bc1, inv_bc2);
    if (wide[i]) {
      *reinterpret_cast<float4*>(p.grads + e[i][0]) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
      if constexpr (OPT != SEG_SGD) *reinterpret_cast<float4*>(p.s1 + e[i][0]) = make_float4(m[i][0], m[i][1], m[i][2], m[i][3]);
      if constexpr (OPT == SEG_ADAM) *reinterpret_cast<float4*>(p.s2 + e[i][0]) = make_float4(v[i][0], v[i][1], v[i][2], v[i][3]);
      *reinterpret_cast<float4*>(p.params + e[i][0]) = make_float4(w[i][0], w[i][1], w[i][2], w[i][3]);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (e[i][j] < 0) continue;
        p.grads[e[i][j]] = acc[i][j];
        if constexpr (OPT != SEG_SGD) p.s1[e[i][j]] = m[i][j];
        if constexpr (OPT == SEG_ADAM) p.s2[e[i][j]] = v[i][j];
        p.params[e[i][j]] = w[i][j];
      }
    }
  }
}

// CTAs the second kernel aims at: two per SM, so that short tiles of different layers overlap.
constexpr int kWgradTargetCtas = 296;

int total_wgrad_tiles(int n_layers, const int* widths) {
  int t = 0;
  for (int l = 0; l < n_layers; ++l) t += wgrad_tiles(widths[l], widths[l + 1]);
  return t;
}

std::atomic<bool> g_smem_attr_set[2][64];    // [R == 16][device]

}  // namespace

bool small_step_supported(int n_layers, const int* widths) {
  if (n_layers < 1 || n_layers > kSmallMaxLayers || widths[0] > kSmallMaxInput) return false;
  for (int l = 1; l <= n_layers; ++l)
    if (widths[l] > kSmallMaxWidth) return false;
  return true;
}

// Rows of the batch per CTA of the first kernel: 8 while that fills the GPU at most once, 16 beyond.
int small_step_rows(int batch) { return batch <= 148 * 8 ? 8 : 16; }

bool small_step_batch_ok(int batch) {
  const int R = small_step_rows(batch);
  return (batch + R - 1) / R <= loss_max_partials();
}

int small_step_wgrad_slots(int n_layers, const int* widths) {
  const int tiles = total_wgrad_tiles(n_layers, widths);
  return tiles * std::max(1, kWgradTargetCtas / tiles);
}

cudaError_t launch_small_fwd_bwd(const SmallStep& p, const float* x, const int32_t* cls, const float* gather,
                                 float* loss_to, cudaStream_t s) {
  const int R = small_step_rows(p.batch);
  const size_t smem = fwd_bwd_smem_floats(p, R) * sizeof(float);
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::atomic<bool>& flag = g_smem_attr_set[R == 16][dev];
  if (!flag.load(std::memory_order_acquire)) {
    // the largest footprint any supported segment has, so that the attribute is set once per device
    const size_t max_floats = (size_t)SS_STAGES * SS_STAGE_FLOATS + 2 * (size_t)kSmallMaxWidth * R +
                              ((size_t)kSmallMaxInput + (size_t)kSmallMaxLayers * kSmallMaxWidth) * R;
    e = R == 16 ? cudaFuncSetAttribute(small_fwd_bwd_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(max_floats * 4))
                : cudaFuncSetAttribute(small_fwd_bwd_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(max_floats * 4));
    if (e != cudaSuccess) return e;
    flag.store(true, std::memory_order_release);
  }
  const int grid = (p.batch + R - 1) / R;
  if (R == 16) launch_k(small_fwd_bwd_kernel<16>, dim3(grid), dim3(SS_THREADS), smem, s, p, x, cls, gather, loss_to);
  else launch_k(small_fwd_bwd_kernel<8>, dim3(grid), dim3(SS_THREADS), smem, s, p, x, cls, gather, loss_to);
  return cudaGetLastError();
}

cudaError_t launch_small_wgrad_update(const SmallStep& p, cudaStream_t s) {
  const int tiles = total_wgrad_tiles(p.n_layers, p.widths);
  // split the batch while that adds CTAs the GPU has room for and leaves every split at least two k-steps
  int splits = std::min(std::min(kWgradTargetCtas / tiles, p.wg_slots / tiles), p.batch / (2 * WK));
  if (splits < 1) splits = 1;
  int k_per_split = ((p.batch + splits - 1) / splits + WK - 1) / WK * WK;
  splits = (p.batch + k_per_split - 1) / k_per_split;
  const int grid = tiles * splits;
  switch (p.optimizer) {
    case SEG_SGD: launch_k(small_wgrad_update_kernel<SEG_SGD>, dim3(grid), dim3(SS_THREADS), 0, s, p, splits, k_per_split); break;
    case SEG_SGD_MOMENTUM: launch_k(small_wgrad_update_kernel<SEG_SGD_MOMENTUM>, dim3(grid), dim3(SS_THREADS), 0, s, p, splits, k_per_split); break;
    case SEG_ADAM: launch_k(small_wgrad_update_kernel<SEG_ADAM>, dim3(grid), dim3(SS_THREADS), 0, s, p, splits, k_per_split); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace segk
