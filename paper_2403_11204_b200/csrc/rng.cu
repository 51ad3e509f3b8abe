// Random streams of the segment trainer: Philox4x32-10 (Salmon et al., SC'11), open-interval
// uniforms, a bit-reproducible standard normal, the synthetic intermediate labels of Eq. 1 and
// the U(-1/sqrt(fan_in), 1/sqrt(fan_in)) Linear initialisation.
//
// Every output element depends only on (seed, segment_id, layer, tag, element index): key =
// (seed lo, seed hi), counter = (q lo, q hi, segment_id, 4*layer + tag) with q = element / 4 and
// the element's word = element mod 4.  The launch geometry never enters the values.
//
// The normal sampler uses integer operations and individually rounded binary64 operations only
// (explicit _rn intrinsics, so the compiler cannot contract them), which makes its output
// identical on every IEEE-754 machine that follows the same written recipe.
#include "common.cuh"

namespace segk {
namespace {

constexpr uint32_t kMulA = 0xD2511F53u, kMulB = 0xCD9E8D57u;
constexpr uint32_t kWeylA = 0x9E3779B9u, kWeylB = 0xBB67AE85u;

__device__ __forceinline__ void philox4x32_10(uint32_t (&c)[4], uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi_a = __umulhi(kMulA, c[0]), lo_a = kMulA * c[0];
    const uint32_t hi_b = __umulhi(kMulB, c[2]), lo_b = kMulB * c[2];
    const uint32_t w0 = hi_b ^ c[1] ^ k0;
    const uint32_t w2 = hi_a ^ c[3] ^ k1;
    c[0] = w0; c[1] = lo_b; c[2] = w2; c[3] = lo_a;
    k0 += kWeylA; k1 += kWeylB;
  }
}

// u = (2*(r >> 9) + 1) * 2^-24: exact in fp32, strictly inside (0,1).
__device__ __forceinline__ float uniform_open01(uint32_t r) {
  return __fmul_rn(__uint2float_rn(2u * (r >> 9) + 1u), 5.9604644775390625e-08f);
}

// ln(n * 2^-24), n odd in [1, 2^24):  n = m 2^e, m in [1,2) folded to (sqrt(1/2), sqrt 2];
// ln m = 2 atanh((m-1)/(m+1)) by its series through s^15.
__device__ __forceinline__ double log_u24(uint32_t n) {
  int e = 31 - __clz(n);
  double m = __dmul_rn(__uint2double_rn(n), __hiloint2double((1023 - e) << 20, 0));  // exact scaling
  if (m > 1.4142135623730951) { m = __dmul_rn(m, 0.5); e += 1; }
  const double s = __ddiv_rn(__dadd_rn(m, -1.0), __dadd_rn(m, 1.0));
  const double z = __dmul_rn(s, s);
  double acc = 2.0 / 15.0;
  acc = __dadd_rn(__dmul_rn(acc, z), 2.0 / 13.0);
  acc = __dadd_rn(__dmul_rn(acc, z), 2.0 / 11.0);
  acc = __dadd_rn(__dmul_rn(acc, z), 2.0 / 9.0);
  acc = __dadd_rn(__dmul_rn(acc, z), 2.0 / 7.0);
  acc = __dadd_rn(__dmul_rn(acc, z), 2.0 / 5.0);
  acc = __dadd_rn(__dmul_rn(acc, z), 2.0 / 3.0);
  acc = __dadd_rn(__dmul_rn(acc, z), 2.0);
  const double p = __dmul_rn(s, acc);
  return __dadd_rn(__dmul_rn(__int2double_rn(e - 24), 0.6931471805599453), p);
}

// cos and sin of 2 pi (j + 0.5) / 2^24 for a 24-bit j: quadrant and octant by integer
// arithmetic, then Taylor polynomials on (0, pi/4).
__device__ __forceinline__ void sincos_u24(uint32_t j, double& c_out, double& s_out) {
  const uint32_t quad = j >> 22;
  const uint32_t t = j & 0x3FFFFFu;
  const bool upper = (t >> 21) != 0u;
  uint32_t tp = t & 0x1FFFFFu;
  if (upper) tp = 0x1FFFFFu - tp;
  // (pi/4) * 2^-21; the power-of-two factor is exact
  const double psi = __dmul_rn(__dadd_rn(__uint2double_rn(tp), 0.5),
                               0.7853981633974483 * 4.76837158203125e-07);
  const double y = __dmul_rn(psi, psi);
  double sp = -1.0 / 1307674368000.0;
  sp = __dadd_rn(__dmul_rn(sp, y), 1.0 / 6227020800.0);
  sp = __dadd_rn(__dmul_rn(sp, y), -1.0 / 39916800.0);
  sp = __dadd_rn(__dmul_rn(sp, y), 1.0 / 362880.0);
  sp = __dadd_rn(__dmul_rn(sp, y), -1.0 / 5040.0);
  sp = __dadd_rn(__dmul_rn(sp, y), 1.0 / 120.0);
  sp = __dadd_rn(__dmul_rn(sp, y), -1.0 / 6.0);
  sp = __dadd_rn(__dmul_rn(sp, y), 1.0);
  double s = __dmul_rn(psi, sp);
  double c = -1.0 / 87178291200.0;
  c = __dadd_rn(__dmul_rn(c, y), 1.0 / 479001600.0);
  c = __dadd_rn(__dmul_rn(c, y), -1.0 / 3628800.0);
  c = __dadd_rn(__dmul_rn(c, y), 1.0 / 40320.0);
  c = __dadd_rn(__dmul_rn(c, y), -1.0 / 720.0);
  c = __dadd_rn(__dmul_rn(c, y), 1.0 / 24.0);
  c = __dadd_rn(__dmul_rn(c, y), -1.0 / 2.0);
  c = __dadd_rn(__dmul_rn(c, y), 1.0);
  if (upper) { const double tmp = s; s = c; c = tmp; }
  switch (quad) {
    case 0: c_out = c;  s_out = s;  break;
    case 1: c_out = -s; s_out = c;  break;
    case 2: c_out = -c; s_out = -s; break;
    default: c_out = s; s_out = -c; break;
  }
}

// Box-Muller on one pair of words.
__device__ __forceinline__ void normal_pair(uint32_t r0, uint32_t r1, float& z0, float& z1) {
  const double rad = __dsqrt_rn(__dmul_rn(-2.0, log_u24(2u * (r0 >> 9) + 1u)));
  double c, s;
  sincos_u24(r1 >> 8, c, s);
  z0 = __double2float_rn(__dmul_rn(rad, c));
  z1 = __double2float_rn(__dmul_rn(rad, s));
}

enum Transform : int { TR_UNIFORM_SCALED = 0, TR_NORMAL = 1, TR_SYMMETRIC = 2 };

// One thread per Philox block (four consecutive elements of the row-major [rows][cols] tensor).
__global__ void __launch_bounds__(256)
fill_random_kernel(float* __restrict__ dst, int64_t n_elems, int cols, int64_t ld, uint32_t k0,
                   uint32_t k1, uint32_t segment_id, uint32_t stream, int transform, float scale) {
  pdl_wait();
  pdl_trigger();
  const int64_t n_blocks = (n_elems + 3) / 4;
  for (int64_t q = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; q < n_blocks;
       q += (int64_t)gridDim.x * blockDim.x) {
    uint32_t c[4] = {(uint32_t)(q & 0xFFFFFFFFll), (uint32_t)(q >> 32), segment_id, stream};
    philox4x32_10(c, k0, k1);
    float v[4];
    if (transform == TR_NORMAL) {
      normal_pair(c[0], c[1], v[0], v[1]);
      normal_pair(c[2], c[3], v[2], v[3]);
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float u = uniform_open01(c[i]);
        v[i] = transform == TR_UNIFORM_SCALED
                   ? __fmul_rn(scale, u)
                   : __fmul_rn(__fadd_rn(__fmul_rn(2.0f, u), -1.0f), scale);
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int64_t e = 4 * q + i;
      if (e < n_elems) dst[(e / cols) * ld + (e % cols)] = v[i];
    }
  }
}

cudaError_t fill(float* dst, int rows, int cols, int64_t ld, uint64_t seed, int segment_id,
                 uint32_t stream, int transform, float scale, cudaStream_t s) {
  const int64_t n = (int64_t)rows * cols;
  if (n == 0) return cudaSuccess;
  const int64_t blocks = ((n + 3) / 4 + 255) / 256;
  const int grid = (int)(blocks < 148 * 8 ? blocks : 148 * 8);
  launch_k(fill_random_kernel, dim3(grid), dim3(256), 0, s, dst, n, cols, ld, (uint32_t)(seed & 0xFFFFFFFFull),
                                          (uint32_t)(seed >> 32), (uint32_t)segment_id, stream,
                                          transform, scale);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_gen_labels(float* dst, int n_classes, int n_p, uint64_t seed, int segment_id,
                              int dist, float kappa, cudaStream_t s) {
  return fill(dst, n_classes, n_p, n_p, seed, segment_id, 0u,
              dist == SEG_LABEL_NORMAL ? TR_NORMAL : TR_UNIFORM_SCALED, kappa, s);
}

cudaError_t launch_init_uniform(float* dst, int rows, int cols, int64_t ld, uint64_t seed,
                                int segment_id, int layer, int tag, float bound, cudaStream_t s) {
  return fill(dst, rows, cols, ld, seed, segment_id, (uint32_t)(4 * layer + tag), TR_SYMMETRIC,
              bound, s);
}

}  // namespace segk
