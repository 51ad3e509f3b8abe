// FFMA matrix products for the fp32 precision mode (tensor cores have no fp32-operand kind), for
// shapes the tensor-core path does not take, and as an on-device cross-check of that path.
// One kernel covers forward (A W^T), dgrad (dZ W) and wgrad (dZ^T A) through element strides.
#include "common.cuh"

namespace segk {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, PAD = 4;

template <typename T>
__device__ __forceinline__ float to_f(T v);
template <>
__device__ __forceinline__ float to_f<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(GemmDesc g) {
  pdl_wait();
  pdl_trigger();
  __shared__ __align__(16) float As[BK][BM + PAD];
  __shared__ __align__(16) float Bs[BK][BN + PAD];
  const TIn* __restrict__ A = reinterpret_cast<const TIn*>(g.A);
  const TIn* __restrict__ B = reinterpret_cast<const TIn*>(g.B);
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const bool a_kfast = (g.a_sk == 1), b_nfast = (g.b_sn == 1);
  float acc[4][4] = {};
  for (int k0 = 0; k0 < g.K; k0 += BK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = threadIdx.x + 256 * i;
      const int k = a_kfast ? (idx & (BK - 1)) : (idx / BM);
      const int m = a_kfast ? (idx / BK) : (idx & (BM - 1));
      float v = 0.f;
      if (m0 + m < g.M && k0 + k < g.K) v = to_f<TIn>(A[(int64_t)(m0 + m) * g.a_sm + (int64_t)(k0 + k) * g.a_sk]);
      As[k][m] = v;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = threadIdx.x + 256 * i;
      const int n = b_nfast ? (idx & (BN - 1)) : (idx / BK);
      const int k = b_nfast ? (idx / BN) : (idx & (BK - 1));
      float v = 0.f;
      if (n0 + n < g.N && k0 + k < g.K) v = to_f<TIn>(B[(int64_t)(k0 + k) * g.b_sk + (int64_t)(n0 + n) * g.b_sn]);
      Bs[k][n] = v;
    }
    __syncthreads();
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

cudaError_t launch_gemm_simt(const GemmDesc& g, cudaStream_t s) {
  if (g.M <= 0 || g.N <= 0) return cudaSuccess;
  if (g.a_dt != g.b_dt) return cudaErrorInvalidValue;
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM);
  if (g.a_dt == DT_F32 && g.c_dt == DT_F32) launch_k(gemm_simt_kernel<float, float>, dim3(grid), dim3(256), 0, s, g);
  else if (g.a_dt == DT_BF16 && g.c_dt == DT_BF16)
    launch_k(gemm_simt_kernel<__nv_bfloat16, __nv_bfloat16>, dim3(grid), dim3(256), 0, s, g);
  else if (g.a_dt == DT_BF16 && g.c_dt == DT_F32)
    launch_k(gemm_simt_kernel<__nv_bfloat16, float>, dim3(grid), dim3(256), 0, s, g);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace segk
