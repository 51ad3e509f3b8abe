// FFMA matrix products for the fp32 precision mode (tensor cores have no fp32-operand kind), for
// shapes the tensor-core path does not take, and as an on-device cross-check of that path.
// One kernel covers forward (A W^T), dgrad (dZ W) and wgrad (dZ^T A) through element strides.
//
// Small layers with a long contraction (the weight gradient of the paper's 80- and 60-wide layers
// over a batch of 1410: one or two output tiles, 88 k-steps) would leave the GPU idle, so K can be
// split over gridDim.z CTAs per tile: every CTA stores its partial tile to a workspace, the last one
// to arrive adds the partials in split order (a fixed order: bit-reproducible), applies the epilogue
// and leaves the arrival counter at zero.
#include <algorithm>

#include "common.cuh"

namespace segk {
namespace {

constexpr int BM = 64, BN = 64, BK = 32, PAD = 4;

template <typename T>
__device__ __forceinline__ float to_f(T v);
template <>
__device__ __forceinline__ float to_f<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(GemmDesc g, int k_per_split) {
  pdl_wait();
  pdl_trigger();
  __shared__ bool is_last;
  __shared__ __align__(16) float As[BK][BM + PAD];
  __shared__ __align__(16) float Bs[BK][BN + PAD];
  const TIn* __restrict__ A = reinterpret_cast<const TIn*>(g.A);
  const TIn* __restrict__ B = reinterpret_cast<const TIn*>(g.B);
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const bool a_kfast = (g.a_sk == 1), b_nfast = (g.b_sn == 1);
  float acc[4][4] = {};
  const int k_begin = blockIdx.z * k_per_split, k_end = min(g.K, k_begin + k_per_split);
  constexpr int LD = BM * BK / 256;          // elements of each operand tile a thread fetches per k-step
  float ra[LD], rb[LD];
  // fetch of one k-step into registers; the next step's fetch is issued before this step's arithmetic
  auto fetch = [&](int k0) {
#pragma unroll
    for (int i = 0; i < LD; ++i) {
      const int idx = threadIdx.x + 256 * i;
      const int k = a_kfast ? (idx & (BK - 1)) : (idx / BM);
      const int m = a_kfast ? (idx / BK) : (idx & (BM - 1));
      ra[i] = 0.f;
      if (m0 + m < g.M && k0 + k < k_end) ra[i] = to_f<TIn>(A[(int64_t)(m0 + m) * g.a_sm + (int64_t)(k0 + k) * g.a_sk]);
    }
#pragma unroll
    for (int i = 0; i < LD; ++i) {
      const int idx = threadIdx.x + 256 * i;
      const int n = b_nfast ? (idx & (BN - 1)) : (idx / BK);
      const int k = b_nfast ? (idx / BN) : (idx & (BK - 1));
      rb[i] = 0.f;
      if (n0 + n < g.N && k0 + k < k_end) rb[i] = to_f<TIn>(B[(int64_t)(k0 + k) * g.b_sk + (int64_t)(n0 + n) * g.b_sn]);
    }
  };
  if (k_begin < k_end) fetch(k_begin);
  for (int k0 = k_begin; k0 < k_end; k0 += BK) {
#pragma unroll
    for (int i = 0; i < LD; ++i) {
      const int idx = threadIdx.x + 256 * i;
      As[a_kfast ? (idx & (BK - 1)) : (idx / BM)][a_kfast ? (idx / BK) : (idx & (BM - 1))] = ra[i];
      Bs[b_nfast ? (idx / BN) : (idx & (BK - 1))][b_nfast ? (idx & (BN - 1)) : (idx / BK)] = rb[i];
    }
    __syncthreads();
    if (k0 + BK < k_end) fetch(k0 + BK);
#pragma unroll
    for (int k = 0; k < BK; ++k) {
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
  if (gridDim.z > 1) {
    const int tile = blockIdx.y * gridDim.x + blockIdx.x;
    float* slot = g.simt_scratch + ((size_t)tile * gridDim.z + blockIdx.z) * kSimtTileFloats;
#pragma unroll
    for (int i = 0; i < 4; ++i)
      *reinterpret_cast<float4*>(slot + (ty * 4 + i) * BN + tx * 4) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(g.simt_counters + tile, 1u) == gridDim.z - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const float* base = g.simt_scratch + (size_t)tile * gridDim.z * kSimtTileFloats;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (unsigned int z = 0; z < gridDim.z; ++z) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float4 p = __ldcg(reinterpret_cast<const float4*>(base + (size_t)z * kSimtTileFloats + (ty * 4 + i) * BN + tx * 4));
        acc[i][0] += p.x; acc[i][1] += p.y; acc[i][2] += p.z; acc[i][3] += p.w;
      }
    }
    if (threadIdx.x == 0) g.simt_counters[tile] = 0u;
  }
  TOut* __restrict__ C = reinterpret_cast<TOut*>(g.C);
  const TOut* __restrict__ mask = reinterpret_cast<const TOut*>(g.mask);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= g.N) continue;
      float v = acc[i][j];
      if (g.epi == EPI_BIAS_ACT) {
        v += g.bias[n];
        if (g.relu) v = fmaxf(v, 0.f);
      } else if (g.epi == EPI_MASK) {
        if (!(to_f<TOut>(mask[(int64_t)m * g.ldmask + n]) > 0.f)) v = 0.f;
      }
      v = apply_round(v, g.c_round);
      if constexpr (sizeof(TOut) == 2) C[(int64_t)m * g.ldc + n] = __float2bfloat16_rn(v);
      else C[(int64_t)m * g.ldc + n] = v;
    }
  }
}

}  // namespace

// Partial tiles the split of an M x N x K product would use with an unlimited workspace (0: no split).
int gemm_simt_slots(int M, int N, int K) {
  const int tiles = ((N + BN - 1) / BN) * ((M + BM - 1) / BM);
  if (tiles < 1 || tiles > 148) return 0;
  const int splits = std::min(148 / tiles, K / (4 * BK));
  return splits > 1 ? tiles * splits : 0;
}

cudaError_t launch_gemm_simt(const GemmDesc& g, cudaStream_t s) {
  if (g.M <= 0 || g.N <= 0) return cudaSuccess;
  if (g.a_dt != g.b_dt) return cudaErrorInvalidValue;
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM);
  // split K while that adds CTAs the GPU has room for and leaves every split at least 4 k-steps
  const int tiles = (int)(grid.x * grid.y);
  int splits = 1;
  if (g.simt_scratch != nullptr && g.simt_counters != nullptr && tiles <= g.simt_slots) {
    splits = std::min(std::min(148 / tiles, g.simt_slots / tiles), g.K / (4 * BK));
    if (splits < 1) splits = 1;
  }
  int k_per_split = ((g.K + splits - 1) / splits + BK - 1) / BK * BK;
  if (k_per_split < BK) k_per_split = BK;
  splits = g.K > 0 ? (g.K + k_per_split - 1) / k_per_split : 1;
  grid.z = (unsigned)std::max(splits, 1);
  if (g.a_dt == DT_F32 && g.c_dt == DT_F32) launch_k(gemm_simt_kernel<float, float>, dim3(grid), dim3(256), 0, s, g, k_per_split);
  else if (g.a_dt == DT_BF16 && g.c_dt == DT_BF16)
    launch_k(gemm_simt_kernel<__nv_bfloat16, __nv_bfloat16>, dim3(grid), dim3(256), 0, s, g, k_per_split);
  else if (g.a_dt == DT_BF16 && g.c_dt == DT_F32)
    launch_k(gemm_simt_kernel<__nv_bfloat16, float>, dim3(grid), dim3(256), 0, s, g, k_per_split);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace segk
