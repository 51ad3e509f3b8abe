// Tensor-core matrix products for sm_100a: TMA -> shared memory -> tcgen05.mma -> TMEM -> epilogue.
//
// One persistent, warp-specialised kernel serves the three products of a Linear layer:
//   forward  C = A W^T     : both operands K-major (contraction index contiguous in memory)
//   dgrad    C = dZ W      : A K-major, B MN-major
//   wgrad    C = dZ^T A    : both operands MN-major (contraction over the batch)
// with bf16 operands (kind::f16) or TF32 operands (kind::tf32) and fp32 accumulation in TMEM.
//
// CTA = 6 warps.  Warp 0 lane 0 issues TMA loads into a ring of shared-memory stages; warp 1 owns
// the TMEM allocation and its lane 0 issues the MMAs; warps 2..5 drain the accumulator (each warp
// reads its own 32 TMEM lanes), apply the epilogue and store.  Two accumulator buffers in TMEM let
// the epilogue of tile i overlap the main loop of tile i+1.
//
// Shared-memory operand tiles use the 128-byte swizzle.  K-major tile: rows of 128 bytes (64 bf16
// or 32 TF32 along K), 8-row groups 1024 bytes apart.  MN-major tile: chunks of 64 bf16 / 32 TF32
// along M or N; inside a chunk each K index is one 128-byte row; chunks follow each other at
// BLOCK_K * 128 bytes.  bf16 MN-major tiles use the ordinary 128-byte swizzle (16-byte atoms,
// 8-row groups 1024 bytes apart); 32-bit MN-major tiles must use the 128-byte swizzle with
// 32-byte atoms (4-row groups 512 bytes apart), in the tensor map and in the descriptor alike.
//
// Small problems (few output tiles, long K) use gemm_tc_splitk_kernel instead: a thread-block
// cluster of 2, 4 or 8 CTAs shares one 128 x 64 output tile, each CTA contracts its own slice of K
// into TMEM, and the partial tiles are combined through distributed shared memory as a
// reduce-scatter (every CTA bulk-copies column slice j of its partial into CTA j's shared memory;
// CTA j adds what it received and runs the epilogue on that slice).  One SM's shared-memory fill rate bounds a single CTA's main loop, so spreading K over a
// cluster shortens exactly the part of the kernel that grows with the problem.
//
// Large problems use gemm_tc_pair_kernel: two CTAs of a cluster share one 256 x 256 output tile
// through tcgen05.mma.cta_group::2.  Each CTA stages its own 128 rows of A and its own 128 columns
// of B (32 KiB per k-block instead of 48 KiB for the same 128 x 256 x 64 of work per SM), which is
// what matters because the single-CTA kernel is bound by one SM's shared-memory fill rate, not by
// the tensor pipe.  The even CTA issues the MMAs for the pair; TMA loads of both CTAs complete on
// the even CTA's "full" barrier; one commit frees the stage in both CTAs.
//
// The persistent kernels (one CTA or a CTA pair per tile) number their tiles in groups of tile rows
// sized so that the operand panels a wave of tiles shares stay in L2 (tile_coords, pick_group_m),
// and store their output through shared memory: each epilogue warp writes its 32 rows x 64 bytes into
// a staging buffer with the 64-byte swizzle and a bulk tensor store writes the box, clipped to the
// matrix (epilogue_store_staged).  Ring plus staging stay within 192 KiB: a larger footprint per CTA
// measured 3-5 % slower over a whole training step although every product alone got faster.
//
// An optional variant of both persistent kernels applies the optimizer update inside the
// weight-gradient product (eight extra warps stream the update of every stored tile).  It measured
// slower than the separate update launch - the operand loads of the main loop already use most of
// what L2 delivers to an SM - and is off unless SEG_FUSED_UPDATE=1.
//
// Every wait on an mbarrier is bounded: after about two seconds the waiting thread raises an abort
// flag, records DEV_TIMEOUT in the status word and all roles leave their loops; TMEM is released
// before the CTA exits.
#include <cuda.h>
#include <stdlib.h>

#include <algorithm>
#include <atomic>
#include <mutex>

#include "common.cuh"

namespace segk {
namespace {

constexpr int BLOCK_M = 128;
constexpr int TILE_ROW_BYTES = 128;                    // one swizzle row
constexpr int A_TILE_BYTES = BLOCK_M * TILE_ROW_BYTES; // 16 KiB per stage
constexpr int NUM_THREADS = 192;                       // TMA warp, MMA warp, four epilogue warps
constexpr int UPDATE_WARPS = 8;                        // fused-update variants: eight more warps stream the optimizer update
constexpr int NUM_THREADS_FUSED = NUM_THREADS + 32 * UPDATE_WARPS;
constexpr int SMEM_BUDGET = 192 * 1024;                // operand ring
constexpr int SMEM_EXTRA = 2048;                       // alignment slack + barriers
// Output staging of the persistent kernels: every epilogue warp owns two buffers of 32 rows x 64 bytes (32 bf16 or 16
// fp32 columns), written with the shared-memory swizzle of the output tensor map and drained by bulk tensor stores, so
// that global memory sees whole 64-byte row segments instead of 32 separate 16-byte pieces.  16 KiB in all, taken out
// of the operand ring's 192 KiB (one stage fewer): the CTA's footprint must not grow.  Measured: with the staging area
// ON TOP of a full ring (210 or 226 KiB per CTA) every product got faster when timed alone (weight gradients by 10 %)
// and every training step 3-5 % SLOWER, and 8 KiB of unused padding alone did the same to the old kernels; within the
// old footprint the steps gain 1-3.5 %.
constexpr int STAGE_OUT_WARP_BYTES = 32 * 64;          // one buffer of one warp
constexpr int STAGE_OUT_BYTES = 4 * 2 * STAGE_OUT_WARP_BYTES;   // 16 KiB
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;

// ---- PTX wrappers ------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when the wait was abandoned (own time-out or another role's abort).
// The product kernels pass the compile-time limit; the self-test kernel passes a short one.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int* dev_status, uint64_t limit_ns = WAIT_LIMIT_NS) {
  uint32_t spins = 0;
  uint64_t t0 = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 0xFFu) == 0u) {
      if (*abort_flag) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) {
        *abort_flag = 1;
        atomicOr(dev_status, (int)DEV_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
// bulk tensor store shared -> global of one box (clipped to the tensor's extent), tracked by the thread's bulk groups
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// at most one of this thread's bulk stores may still be reading its shared-memory source
__device__ __forceinline__ void tma_store_wait_source_but_one() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
// all of this thread's bulk stores are complete
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
template <bool TF32>
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  if constexpr (TF32) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
  }
}
// 32 lanes x 32 columns of fp32: thread i of the warp receives row (lane base + i), 32 columns.
__device__ __forceinline__ void tmem_load_32x32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor (sm_100 format): start address, leading / stride byte offsets
// in 16-byte units, descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes,
                                                   uint32_t layout_type) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version
  d |= (uint64_t)layout_type << 61;   // 2: 128-byte swizzle; 1: 128-byte swizzle, 32-byte atoms
  return d;
}

// Tile order of the persistent kernels.  Tiles are numbered in groups of `group_m` rows of tiles: inside a
// group the row index runs fastest, then the column index, and the groups follow each other.  The CTAs (or pairs)
// work on consecutive tile numbers at the same time and sweep K in step, so a wave covers group_m row blocks by
// (CTAs / group_m) column blocks; the row blocks' operand panels (group_m x tile rows x K) are what consecutive
// waves share and must survive in L2 while the column blocks' panels stream through.  group_m = all rows of tiles
// is the plain row-fastest order.
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int group_m, int& m_idx, int& n_idx) {
  const int per_group = group_m * tiles_n;
  const int group = t / per_group, r = t - group * per_group;
  const int first_m = group * group_m;
  const int gsize = min(group_m, tiles_m - first_m);
  n_idx = r / gsize;
  m_idx = first_m + (r - n_idx * gsize);
}

struct EpilogueArgs {
  void* C;
  int64_t ldc;
  int c_dt, c_round, epi, relu;
  const float* bias;
  const void* mask;
  int64_t ldmask;
  int staged;               // persistent kernels: store C through shared memory and bulk tensor stores
  LossFuse loss;
  FusedUpdate upd;
};

template <int BLOCK_N>
struct SmemLayout {
  static constexpr int B_TILE_BYTES = BLOCK_N * TILE_ROW_BYTES;
  static constexpr int STAGE_BYTES = A_TILE_BYTES + B_TILE_BYTES;
  static constexpr int STAGES = (SMEM_BUDGET / STAGE_BYTES) > 8 ? 8 : (SMEM_BUDGET / STAGE_BYTES);   // without staging
  // with the output staging area inside the same budget (ring + staging stay within 192 KiB, see STAGE_OUT_BYTES)
  static constexpr int STAGES_STAGED = ((SMEM_BUDGET - STAGE_OUT_BYTES) / STAGE_BYTES) > 8 ? 8 : ((SMEM_BUDGET - STAGE_OUT_BYTES) / STAGE_BYTES);
  static constexpr int TOTAL = STAGES * STAGE_BYTES + SMEM_EXTRA;                                        // upper bound of both layouts
};

// Side inputs of the epilogue for up to 32 consecutive columns of one row: the bias values (forward)
// or the stored activations that give the ReLU mask (dgrad; bf16 activations packed two per word).
// They do not depend on the accumulator, so they are fetched before it is waited for and their
// global-memory latency is off the critical path.
struct EpiSide { uint32_t w[32]; };

template <int NV = 32>
__device__ __forceinline__ void epilogue_prefetch(const EpilogueArgs& e, EpiSide& s, int row, bool row_ok,
                                                  int col0, int n_total) {
  const int n_valid = min(NV, n_total - col0);
  if (n_valid <= 0) return;
  const bool whole = (n_valid & 7) == 0;
  if (e.epi == EPI_BIAS_ACT) {
    const float* brow = e.bias + col0;
    if (whole && ((reinterpret_cast<uintptr_t>(brow) & 15u) == 0)) {
#pragma unroll
      for (int j = 0; j < NV; j += 4) {
        if (j < n_valid) {
          const uint4 b = __ldg(reinterpret_cast<const uint4*>(brow + j));
          s.w[j] = b.x; s.w[j + 1] = b.y; s.w[j + 2] = b.z; s.w[j + 3] = b.w;
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < NV; ++j) if (j < n_valid) s.w[j] = __float_as_uint(__ldg(brow + j));
    }
  } else if (e.epi == EPI_MASK && row_ok) {
    if (e.c_dt == DT_BF16) {
      const unsigned short* mrow = reinterpret_cast<const unsigned short*>(e.mask) + (int64_t)row * e.ldmask + col0;
      if (whole && ((reinterpret_cast<uintptr_t>(mrow) & 15u) == 0)) {
#pragma unroll
        for (int j = 0; j < NV; j += 8) {
          if (j < n_valid) {
            const uint4 q = __ldg(reinterpret_cast<const uint4*>(mrow + j));
            s.w[j / 2] = q.x; s.w[j / 2 + 1] = q.y; s.w[j / 2 + 2] = q.z; s.w[j / 2 + 3] = q.w;
          }
        }
      } else {
#pragma unroll
        for (int j = 0; j < NV; j += 2) {
          uint32_t lo = 0u, hi = 0u;
          if (j < n_valid) lo = __ldg(mrow + j);
          if (j + 1 < n_valid) hi = __ldg(mrow + j + 1);
          s.w[j / 2] = lo | (hi << 16);
        }
      }
    } else {
      const float* mrow = reinterpret_cast<const float*>(e.mask) + (int64_t)row * e.ldmask + col0;
      if (whole && ((reinterpret_cast<uintptr_t>(mrow) & 15u) == 0)) {
#pragma unroll
        for (int j = 0; j < NV; j += 4) {
          if (j < n_valid) {
            const uint4 m = __ldg(reinterpret_cast<const uint4*>(mrow + j));
            s.w[j] = m.x; s.w[j + 1] = m.y; s.w[j + 2] = m.z; s.w[j + 3] = m.w;
          }
        }
      } else {
#pragma unroll
        for (int j = 0; j < NV; ++j) if (j < n_valid) s.w[j] = __float_as_uint(__ldg(mrow + j));
      }
    }
  }
}

// Epilogue for up to 32 consecutive columns of one row, with the side inputs already in registers.
// Columns are stored in groups of 8 with 16-byte accesses when the group count is whole and the
// row segment is 16-byte aligned (every lane touches its own row, so wide accesses are what keeps
// the number of memory wavefronts down); ragged or unaligned segments fall back to scalar stores.
template <int NV>
__device__ __forceinline__ void epilogue_values(const EpilogueArgs& e, float (&v)[NV], const EpiSide& s, int col0,
                                                int n_total) {
  const int n_valid = min(NV, n_total - col0);
  if (e.epi == EPI_BIAS_ACT) {
#pragma unroll
    for (int j = 0; j < NV; ++j) if (j < n_valid) v[j] += __uint_as_float(s.w[j]);
    if (e.relu) {
#pragma unroll
      for (int j = 0; j < NV; ++j) v[j] = fmaxf(v[j], 0.f);
    }
  } else if (e.epi == EPI_MASK) {
    if (e.c_dt == DT_BF16) {
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        // a bf16 is positive iff its sign bit is clear and it is not zero
        const uint32_t bits = (s.w[j >> 1] >> (16 * (j & 1))) & 0xFFFFu;
        if (j < n_valid && !(bits != 0u && bits < 0x8000u)) v[j] = 0.f;
      }
    } else {
#pragma unroll
      for (int j = 0; j < NV; ++j)
        if (j < n_valid && !(__uint_as_float(s.w[j]) > 0.f)) v[j] = 0.f;
    }
  }
  if (e.c_round == RND_TF32) {
#pragma unroll
    for (int j = 0; j < NV; ++j) v[j] = round_tf32_rne(v[j]);
  }
}

// Stores up to 32 consecutive columns of one row into a [rows][ld] matrix of dtype dt.
template <int NV>
__device__ __forceinline__ void store_row_segment(void* base, int dt, int64_t ld, const float (&v)[NV], int row,
                                                  int col0, int n_total) {
  const int n_valid = min(NV, n_total - col0);
  const bool whole = (n_valid & 7) == 0;
  if (dt == DT_BF16) {
    __nv_bfloat16* crow = reinterpret_cast<__nv_bfloat16*>(base) + (int64_t)row * ld + col0;
    if (whole && ((reinterpret_cast<uintptr_t>(crow) & 15u) == 0)) {
#pragma unroll
      for (int j = 0; j < NV; j += 8) {
        if (j < n_valid) {
          uint4 q;
          __nv_bfloat162 p0 = __floats2bfloat162_rn(v[j], v[j + 1]);
          __nv_bfloat162 p1 = __floats2bfloat162_rn(v[j + 2], v[j + 3]);
          __nv_bfloat162 p2 = __floats2bfloat162_rn(v[j + 4], v[j + 5]);
          __nv_bfloat162 p3 = __floats2bfloat162_rn(v[j + 6], v[j + 7]);
          q.x = *reinterpret_cast<uint32_t*>(&p0); q.y = *reinterpret_cast<uint32_t*>(&p1);
          q.z = *reinterpret_cast<uint32_t*>(&p2); q.w = *reinterpret_cast<uint32_t*>(&p3);
          *reinterpret_cast<uint4*>(crow + j) = q;
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < NV; ++j) if (j < n_valid) crow[j] = __float2bfloat16_rn(v[j]);
    }
  } else {
    float* crow = reinterpret_cast<float*>(base) + (int64_t)row * ld + col0;
    if (whole && ((reinterpret_cast<uintptr_t>(crow) & 15u) == 0)) {
#pragma unroll
      for (int j = 0; j < NV; j += 4) {
        if (j < n_valid) *reinterpret_cast<float4*>(crow + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < NV; ++j) if (j < n_valid) crow[j] = v[j];
    }
  }
}

template <int NV>
__device__ __forceinline__ void epilogue_store(const EpilogueArgs& e, float (&v)[NV], const EpiSide& s, int row,
                                               int col0, int n_total) {
  epilogue_values(e, v, s, col0, n_total);
  store_row_segment(e.C, e.c_dt, e.ldc, v, row, col0, n_total);
}

// The same epilogue through shared memory: the lane's 32 columns go to row `lane` of the warp's staging buffers, 64 bytes
// per row and buffer (all 32 bf16 columns, or 16 fp32 columns: an fp32 chunk takes both buffers), in 16-byte pieces,
// piece j of row r at position j ^ ((r >> 1) & 3) - the 64-byte swizzle, which the output tensor map expects and which
// makes the warp's stores conflict-free - and one bulk tensor store per buffer writes the 32-row box; rows and columns
// beyond the matrix are clipped by the store.  Before a buffer is written, the store issued from it two stores earlier
// has finished reading it (at most one store is left pending).
__device__ __forceinline__ void epilogue_store_staged(const EpilogueArgs& e, const CUtensorMap* map_c, uint8_t* warp_stage,
                                                      float (&v)[32], const EpiSide& s, int lane, int row0, int col0,
                                                      int n_total, int n_rows, int chunk) {
  epilogue_values(e, v, s, col0, n_total);
  const int x = (lane >> 1) & 3;
  if (e.c_dt == DT_BF16) {
    uint8_t* buf = warp_stage + (chunk & 1) * STAGE_OUT_WARP_BYTES;
    if (lane == 0) tma_store_wait_source_but_one();
    __syncwarp();
    uint8_t* rowp = buf + lane * 64;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      __nv_bfloat162 p0 = __floats2bfloat162_rn(v[8 * j], v[8 * j + 1]);
      __nv_bfloat162 p1 = __floats2bfloat162_rn(v[8 * j + 2], v[8 * j + 3]);
      __nv_bfloat162 p2 = __floats2bfloat162_rn(v[8 * j + 4], v[8 * j + 5]);
      __nv_bfloat162 p3 = __floats2bfloat162_rn(v[8 * j + 6], v[8 * j + 7]);
      uint4 q;
      q.x = *reinterpret_cast<uint32_t*>(&p0); q.y = *reinterpret_cast<uint32_t*>(&p1);
      q.z = *reinterpret_cast<uint32_t*>(&p2); q.w = *reinterpret_cast<uint32_t*>(&p3);
      *reinterpret_cast<uint4*>(rowp + ((j ^ x) << 4)) = q;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // generic writes -> visible to the bulk store
    __syncwarp();
    if (lane == 0 && row0 < n_rows) tma_store_2d(map_c, smem_u32(buf), col0, row0);
  } else {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      if (col0 + 16 * h >= n_total) break;                              // uniform: nothing of this half is inside the matrix
      uint8_t* buf = warp_stage + h * STAGE_OUT_WARP_BYTES;
      if (lane == 0) tma_store_wait_source_but_one();
      __syncwarp();
      uint8_t* rowp = buf + lane * 64;
#pragma unroll
      for (int j = 0; j < 4; ++j)
        *reinterpret_cast<float4*>(rowp + ((j ^ x) << 4)) =
            make_float4(v[16 * h + 4 * j], v[16 * h + 4 * j + 1], v[16 * h + 4 * j + 2], v[16 * h + 4 * j + 3]);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0 && row0 < n_rows) tma_store_2d(map_c, smem_u32(buf), col0 + 16 * h, row0);
    }
  }
}

// ---- fused loss (last forward product of a non-final segment) -----------------------------------
__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// Targets of n_cols (<= 32) consecutive columns of one row: row cls[row] of the label matrix, whose
// pitch is n_p.  Fetched ahead of the accumulator like the other side inputs.
template <int NV = 32>
__device__ __forceinline__ void loss_prefetch_target(const LossFuse& l, EpiSide& t, int row, bool row_ok, int col0,
                                                     int n_cols, int n_p) {
  if (n_cols <= 0 || !row_ok) return;
  const float* trow = l.sil + (int64_t)__ldg(l.cls + row) * n_p + col0;
  if (((n_cols & 3) == 0) && ((reinterpret_cast<uintptr_t>(trow) & 15u) == 0)) {
#pragma unroll
    for (int j = 0; j < NV; j += 4) {
      if (j < n_cols) {
        const uint4 q = __ldg(reinterpret_cast<const uint4*>(trow + j));
        t.w[j] = q.x; t.w[j + 1] = q.y; t.w[j + 2] = q.z; t.w[j + 3] = q.w;
      }
    }
  } else {
#pragma unroll
    for (int j = 0; j < NV; ++j) if (j < n_cols) t.w[j] = __float_as_uint(__ldg(trow + j));
  }
}

// Mean-squared-error part of the epilogue for columns [col0, n_end): stores the output, then
// dZ = gscale (a - t) [a > 0], and adds (a - t)^2 to the thread's loss sum; a is the output as it
// is stored (after rounding to the storage type).
template <int NV>
__device__ __forceinline__ void epilogue_store_mse(const EpilogueArgs& e, float (&v)[NV], const EpiSide& s,
                                                   const EpiSide& t, int row, int col0, int n_end, float& lacc) {
  epilogue_values(e, v, s, col0, n_end);
  store_row_segment(e.C, e.c_dt, e.ldc, v, row, col0, n_end);
  const int n_valid = min(NV, n_end - col0);
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    if (j < n_valid) {
      const float a = (e.c_dt == DT_BF16) ? round_bf16_rne(v[j]) : v[j];
      const float d = a - __uint_as_float(t.w[j]);
      lacc = fmaf(d, d, lacc);
      float g = d * e.loss.gscale;
      if (e.loss.relu_mask && !(a > 0.f)) g = 0.f;
      v[j] = apply_round(g, e.loss.dz_round);
    }
  }
  store_row_segment(e.loss.dz, e.loss.dz_dt, e.loss.ld_dz, v, row, col0, n_end);
}

// End of a CTA's epilogue: the four epilogue warps leave their loss sums in shared memory; the last
// warp to arrive adds them in warp order and publishes the CTA's partial; the last CTA of the grid
// adds all partials in index order (a fixed order: bit-reproducible) and writes the batch loss.
// No barrier is used, so a warp that gave up a bounded wait cannot block the others.
__device__ __forceinline__ void loss_finish(const LossFuse& l, float lacc, int quarter, int lane, volatile float* slots,
                                            unsigned int* warp_counter) {
  const float w = warp_sum_f(lacc);
  unsigned int prev = 0;
  if (lane == 0) {
    slots[quarter] = w;
    __threadfence_block();
    prev = atomicAdd(warp_counter, 1u);
  }
  prev = __shfl_sync(0xFFFFFFFFu, prev, 0);
  if (prev != 3u) return;
  __threadfence_block();
  unsigned int done = 0;
  if (lane == 0) {
    const float block_total = ((slots[0] + slots[1]) + slots[2]) + slots[3];
    l.partials[blockIdx.x] = block_total;
    __threadfence();
    done = atomicAdd(l.counter, 1u);
  }
  done = __shfl_sync(0xFFFFFFFFu, done, 0);
  if (done != gridDim.x - 1) return;
  __threadfence();
  float part = 0.f;
  for (unsigned int i = lane; i < gridDim.x; i += 32) part += __ldcg(l.partials + i);
  const float total = warp_sum_f(part);
  if (lane == 0) {
    float* dst = *l.loss_dst;
    if (dst) *dst = total * l.loss_scale;
    *l.counter = 0u;
  }
}

// ---- optimizer update fused into the weight-gradient product ------------------------------------
// Epilogue warps -> update warps of the same CTA: "one more warp has stored its part of a tile".  The
// stores are fenced to device scope before the count moves, the update warps read the gradient with
// L2 loads, so they see it.  The wait is bounded like every other wait of these kernels.
__device__ __forceinline__ void tile_stored_signal(unsigned int* tiles_done, int lane) {
  __threadfence();
  __syncwarp();
  if (lane == 0) atomicAdd(tiles_done, 1u);
}
__device__ __forceinline__ bool tile_stored_wait(volatile unsigned int* tiles_done, unsigned int needed,
                                                 volatile int* abort_flag, int* dev_status, int lane) {
  int ok = 1;
  if (lane == 0) {
    uint32_t spins = 0;
    uint64_t t0 = 0;
    while (*tiles_done < needed) {
      if ((++spins & 0x3Fu) == 0u) {
        if (*abort_flag) { ok = 0; break; }
        const uint64_t now = global_timer_ns();
        if (t0 == 0) t0 = now;
        else if (now - t0 > WAIT_LIMIT_NS) {
          *abort_flag = 1;
          atomicOr(dev_status, (int)DEV_TIMEOUT);
          ok = 0;
          break;
        }
        __nanosleep(200);
      }
    }
  }
  ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
  __threadfence();
  return ok != 0;
}

__device__ __forceinline__ void opt_apply(const FusedUpdate& f, float& p, float g, float& m, float& v,
                                          float inv_bc1, float inv_bc2) {
  switch (f.optimizer) {
    case SEG_SGD: opt_step<SEG_SGD>(p, g, m, v, f, inv_bc1, inv_bc2); break;
    case SEG_SGD_MOMENTUM: opt_step<SEG_SGD_MOMENTUM>(p, g, m, v, f, inv_bc1, inv_bc2); break;
    default: opt_step<SEG_ADAM>(p, g, m, v, f, inv_bc1, inv_bc2); break;
  }
}

// The update of the 128 x TILE_N block of the weight tensor whose gradient sits at g (row pitch ld, as the
// master weights, the optimizer state and the operand copy), rows m0.., columns n0..  Eight warps; a lane
// handles four consecutive columns per access (16 bytes; padding columns up to the pitch hold zeros on
// every side and stay zero), consecutive lanes consecutive groups, and four such groups are in flight per
// lane before the first is used.  Everything is touched once per step: streaming loads and stores, so that
// the operand tiles of the product keep their place in L2.
template <int TILE_N>
__device__ __forceinline__ void update_tile(const FusedUpdate& f, const float* g, int64_t ld, int m0, int n0,
                                            int M, int N, int uw, int lane, float inv_bc1, float inv_bc2) {
  constexpr int VPR = TILE_N / 4;                      // 16-byte groups per tile row
  constexpr int TOTAL = BLOCK_M * VPR;
  constexpr int R = 4;
  constexpr int STRIDE = UPDATE_WARPS * 32;
  const int n_lim = (N + 3) & ~3;                      // <= ld
  const bool adam = f.optimizer == SEG_ADAM, mom = f.optimizer != SEG_SGD;
  for (int base = uw * 32 + lane; base < TOTAL; base += STRIDE * R) {
    float4 G[R], P[R], S1[R], S2[R];
    int64_t off[R];
    bool ok[R];
#pragma unroll
    for (int i = 0; i < R; ++i) {
      const int v = base + i * STRIDE;
      const int row = m0 + v / VPR, c = n0 + (v % VPR) * 4;
      ok[i] = (v < TOTAL) && (row < M) && (c < n_lim);
      off[i] = (int64_t)row * ld + c;
      if (ok[i]) {
        G[i] = __ldcg(reinterpret_cast<const float4*>(g + off[i]));
        P[i] = __ldcs(reinterpret_cast<const float4*>(f.p + off[i]));
        if (mom) S1[i] = __ldcs(reinterpret_cast<const float4*>(f.s1 + off[i]));
        if (adam) S2[i] = __ldcs(reinterpret_cast<const float4*>(f.s2 + off[i]));
      }
    }
#pragma unroll
    for (int i = 0; i < R; ++i) {
      if (!ok[i]) continue;
      float pv[4] = {P[i].x, P[i].y, P[i].z, P[i].w};
      const float gv[4] = {G[i].x, G[i].y, G[i].z, G[i].w};
      float mv[4] = {0.f, 0.f, 0.f, 0.f}, vv[4] = {0.f, 0.f, 0.f, 0.f};
      if (mom) { mv[0] = S1[i].x; mv[1] = S1[i].y; mv[2] = S1[i].z; mv[3] = S1[i].w; }
      if (adam) { vv[0] = S2[i].x; vv[1] = S2[i].y; vv[2] = S2[i].z; vv[3] = S2[i].w; }
#pragma unroll
      for (int k = 0; k < 4; ++k) opt_apply(f, pv[k], gv[k], mv[k], vv[k], inv_bc1, inv_bc2);
      if (mom) __stcs(reinterpret_cast<float4*>(f.s1 + off[i]), make_float4(mv[0], mv[1], mv[2], mv[3]));
      if (adam) __stcs(reinterpret_cast<float4*>(f.s2 + off[i]), make_float4(vv[0], vv[1], vv[2], vv[3]));
      __stcs(reinterpret_cast<float4*>(f.p + off[i]), make_float4(pv[0], pv[1], pv[2], pv[3]));
      if (f.op_dt == DT_BF16) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(pv[0], pv[1]);
        __nv_bfloat162 hi = __floats2bfloat162_rn(pv[2], pv[3]);
        uint2 packed;
        packed.x = *reinterpret_cast<uint32_t*>(&lo);
        packed.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(f.p_op) + off[i]) = packed;
      } else {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(f.p_op) + off[i]) =
            make_float4(apply_round(pv[0], f.op_round), apply_round(pv[1], f.op_round),
                        apply_round(pv[2], f.op_round), apply_round(pv[3], f.op_round));
      }
    }
  }
}

template <bool TF32, bool A_MN, bool B_MN, int BLOCK_N, bool FUSED = false>
__global__ void __launch_bounds__(FUSED ? NUM_THREADS_FUSED : NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_c, int M, int N, int K, EpilogueArgs epi, int* dev_status, int group_m,
               int n_stages) {
  using L = SmemLayout<BLOCK_N>;
  const int STAGES = n_stages;
  constexpr int BLOCK_K = TF32 ? 32 : 64;          // elements per stage along K (128 bytes K-major)
  constexpr int UMMA_K = TF32 ? 8 : 16;            // elements per MMA along K (32 bytes)
  constexpr int CHUNK = TF32 ? 32 : 64;            // elements per 128-byte row along M/N (MN-major)
  constexpr int MN_CHUNK_BYTES = BLOCK_K * TILE_ROW_BYTES;
  constexpr uint32_t TMEM_COLS = 2 * BLOCK_N;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + STAGES * A_TILE_BYTES;
  uint8_t* stage_out = smem + STAGES * L::STAGE_BYTES;                 // 1024-byte aligned: the ring is a multiple of 1 KiB
  uint64_t* bars = reinterpret_cast<uint64_t*>(stage_out + (epi.staged ? STAGE_OUT_BYTES : 0));
  // bars[0..S) full, [S..2S) empty, [2S..2S+2) tmem_full, [2S+2..2S+4) tmem_empty
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  unsigned int* tiles_done = reinterpret_cast<unsigned int*>(tmem_slot + 2);   // FUSED: epilogue-warp arrivals

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };

  if (threadIdx.x == 0) {
    prefetch_tensormap(&map_a);       // descriptor fetch overlaps the rest of the prologue
    prefetch_tensormap(&map_b);
    prefetch_tensormap(&map_c);
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
    *abort_flag = 0;
    *tiles_done = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // index arithmetic (several integer divisions), the first tile's coordinates included: ahead of the dependency wait
  const int tiles_m = (M + BLOCK_M - 1) / BLOCK_M;
  const int tiles_n = (N + BLOCK_N - 1) / BLOCK_N;
  const int n_tiles = tiles_m * tiles_n;
  const int num_k = (K + BLOCK_K - 1) / BLOCK_K;
  int first_m = 0, first_n = 0;
  if ((int)blockIdx.x < n_tiles) tile_coords((int)blockIdx.x, tiles_m, tiles_n, group_m, first_m, first_n);
  pdl_wait();                         // everything above overlapped the previous kernel's tail
  pdl_trigger();

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int fills = 0;                     // stages filled so far, counted up to the ring's depth: the first pass waits for nothing
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
        int m_idx, n_idx;
        if (t == (int)blockIdx.x) { m_idx = first_m; n_idx = first_n; } else tile_coords(t, tiles_m, tiles_n, group_m, m_idx, n_idx);
        const int m0 = m_idx * BLOCK_M, n0 = n_idx * BLOCK_N;
        for (int kb = 0; kb < num_k; ++kb) {
          if (fills < STAGES) ++fills;
          else if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, dev_status)) { ok = false; break; }
          mbar_arrive_expect_tx(full_bar(stage), (uint32_t)L::STAGE_BYTES);
          const uint32_t a_dst = smem_u32(smem_a + stage * A_TILE_BYTES);
          const uint32_t b_dst = smem_u32(smem_b + stage * L::B_TILE_BYTES);
          const int k0 = kb * BLOCK_K;
          if constexpr (A_MN) {
#pragma unroll
            for (int c = 0; c < BLOCK_M / CHUNK; ++c)
              tma_load_2d(a_dst + c * MN_CHUNK_BYTES, &map_a, m0 + c * CHUNK, k0, full_bar(stage));
          } else {
            tma_load_2d(a_dst, &map_a, k0, m0, full_bar(stage));
          }
          if constexpr (B_MN) {
#pragma unroll
            for (int c = 0; c < BLOCK_N / CHUNK; ++c)
              tma_load_2d(b_dst + c * MN_CHUNK_BYTES, &map_b, n0 + c * CHUNK, k0, full_bar(stage));
          } else {
            tma_load_2d(b_dst, &map_b, k0, n0, full_bar(stage));
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      // instruction descriptor: fp32 accumulate, operand format, operand majors, N, M
      constexpr uint32_t fmt = TF32 ? 2u : 1u;
      constexpr uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((A_MN ? 1u : 0u) << 15) |
                                 ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(BLOCK_N >> 3) << 17) |
                                 ((uint32_t)(BLOCK_M >> 4) << 24);
      constexpr uint32_t a_lbo = A_MN ? MN_CHUNK_BYTES : 16, b_lbo = B_MN ? MN_CHUNK_BYTES : 16;
      constexpr uint32_t a_kstep = A_MN ? UMMA_K * TILE_ROW_BYTES : 32;
      constexpr uint32_t b_kstep = B_MN ? UMMA_K * TILE_ROW_BYTES : 32;
      // 32-bit MN-major operands: 32-byte-atom swizzle, groups of 4 K rows (512 bytes)
      constexpr uint32_t a_sbo = (TF32 && A_MN) ? 512 : 1024, b_sbo = (TF32 && B_MN) ? 512 : 1024;
      constexpr uint32_t a_lay = (TF32 && A_MN) ? 1 : 2, b_lay = (TF32 && B_MN) ? 1 : 2;
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, dev_status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BLOCK_N);
        for (int kb = 0; kb < num_k; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, dev_status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = smem_u32(smem_a + stage * A_TILE_BYTES);
          const uint32_t b_src = smem_u32(smem_b + stage * L::B_TILE_BYTES);
#pragma unroll
          for (int kk = 0; kk < BLOCK_K / UMMA_K; ++kk) {
            const uint64_t da = make_smem_desc(a_src + kk * a_kstep, a_lbo, a_sbo, a_lay);
            const uint64_t db = make_smem_desc(b_src + kk * b_kstep, b_lbo, b_sbo, b_lay);
            tc_mma<TF32>(d_tmem, da, db, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          }
          tc_commit(empty_bar(stage));     // frees the stage once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull_bar(acc));         // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp < NUM_THREADS / 32) {
    // ---------------- epilogue warps ----------------
    const int quarter = warp & 3;          // TMEM lanes 32*quarter .. +31 belong to this warp
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
      int m_idx, n_idx;
      if (t == (int)blockIdx.x) { m_idx = first_m; n_idx = first_n; } else tile_coords(t, tiles_m, tiles_n, group_m, m_idx, n_idx);
      const int m0 = m_idx * BLOCK_M, n0 = n_idx * BLOCK_N;
      const int row = m0 + quarter * 32 + lane;
      EpiSide side, side_next;
      epilogue_prefetch(epi, side, row, row < M, n0, N);   // before the wait: latency off the critical path
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, dev_status)) { ok = false; break; }
      tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < BLOCK_N / 32; ++c) {
        const int col0 = n0 + c * 32;
        if (col0 >= N) break;              // uniform across the CTA
        if (c + 1 < BLOCK_N / 32) epilogue_prefetch(epi, side_next, row, row < M, col0 + 32, N);
        float v[32];
        tmem_load_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BLOCK_N + c * 32), v);
        if (FUSED || !epi.staged) {        // (the update warps read the tile back with ordinary loads: ordinary stores)
          if (row < M) epilogue_store(epi, v, side, row, col0, N);
        } else {
          epilogue_store_staged(epi, &map_c, stage_out + quarter * 2 * STAGE_OUT_WARP_BYTES, v, side, lane,
                                m0 + quarter * 32, col0, N, M, c);
        }
        side = side_next;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      if constexpr (FUSED) tile_stored_signal(tiles_done, lane);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) tma_store_wait_all();   // the staging buffers are read, and the output written, before the CTA leaves
  } else if constexpr (FUSED) {
    // ---------------- update warps: the optimizer on every tile this CTA has stored ----------------
    if (warp >= NUM_THREADS / 32) {
      const int uw = warp - NUM_THREADS / 32;
      float inv_bc1 = 1.0f, inv_bc2 = 1.0f;
      if (epi.upd.optimizer == SEG_ADAM) { inv_bc1 = 1.0f / __ldg(epi.upd.bc); inv_bc2 = 1.0f / __ldg(epi.upd.bc + 1); }
      unsigned int needed = 0;
      for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        needed += 4u;
        if (!tile_stored_wait(tiles_done, needed, abort_flag, dev_status, lane)) break;
        int m_idx, n_idx;
        if (t == (int)blockIdx.x) { m_idx = first_m; n_idx = first_n; } else tile_coords(t, tiles_m, tiles_n, group_m, m_idx, n_idx);
        const int m0 = m_idx * BLOCK_M, n0 = n_idx * BLOCK_N;
        update_tile<BLOCK_N>(epi.upd, reinterpret_cast<const float*>(epi.C), epi.ldc, m0, n0, M, N, uw, lane,
                             inv_bc1, inv_bc2);
      }
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  if (*abort_flag) {
    // give copies and MMAs still in flight time to land before shared memory and TMEM are released
    for (int i = 0; i < 64; ++i) __nanosleep(20000);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
}


// ---- cluster helpers (split-K kernel) -----------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
  uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank)); return r;
}
// bulk copy from this CTA's shared memory into a peer's; completes (by bytes) on the peer's mbarrier
__device__ __forceinline__ void bulk_copy_to_peer(uint32_t dst_cluster_addr, uint32_t src_local_addr,
                                                  uint32_t bytes, uint32_t bar_cluster_addr) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_cluster_addr), "r"(src_local_addr), "r"(bytes), "r"(bar_cluster_addr) : "memory");
}
constexpr int SPLITK_BLOCK_N = 64;
constexpr int SPLITK_STAGES = 6;
constexpr int SPLITK_STAGE_BYTES = A_TILE_BYTES + SPLITK_BLOCK_N * TILE_ROW_BYTES;       // 24 KiB
constexpr int SPLITK_RECV_BYTES = 8 * (SPLITK_BLOCK_N / 8) * BLOCK_M * 4;                // [src][col in slice][row] fp32, 32 KiB
constexpr int SPLITK_SMEM = SPLITK_STAGES * SPLITK_STAGE_BYTES + 2 * SPLITK_RECV_BYTES + SMEM_EXTRA;   // + send buffer

// One 128 x 64 output tile per cluster; CTA r of the cluster contracts k-blocks [r*kpc, (r+1)*kpc).
template <bool TF32, bool A_MN, bool B_MN, int SPLIT, bool LOSS = false>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_splitk_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                      int M, int N, int K, EpilogueArgs epi, int* dev_status) {
  constexpr int split = SPLIT;                             // CTAs per cluster
  constexpr int W = SPLITK_BLOCK_N / SPLIT;                // columns of the tile each CTA owns after the exchange
  static_assert(W == 32 || W == 16 || W == 8, "slice width");
  constexpr int BLOCK_N = SPLITK_BLOCK_N;
  constexpr int STAGES = SPLITK_STAGES;
  constexpr int B_TILE_BYTES = BLOCK_N * TILE_ROW_BYTES;
  constexpr int BLOCK_K = TF32 ? 32 : 64;
  constexpr int UMMA_K = TF32 ? 8 : 16;
  constexpr int CHUNK = TF32 ? 32 : 64;
  constexpr int MN_CHUNK_BYTES = BLOCK_K * TILE_ROW_BYTES;
  constexpr uint32_t TMEM_COLS = BLOCK_N;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + STAGES * A_TILE_BYTES;
  float* recv = reinterpret_cast<float*>(smem + STAGES * SPLITK_STAGE_BYTES);                      // [src][col in slice][row]
  float* send = reinterpret_cast<float*>(smem + STAGES * SPLITK_STAGE_BYTES + SPLITK_RECV_BYTES);  // [dest][col in slice][row]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * SPLITK_STAGE_BYTES + 2 * SPLITK_RECV_BYTES);
  // bars[0..S) full, [S..2S) empty, [2S] accumulator complete, [2S+1] partial slices received
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile float* loss_slots = reinterpret_cast<volatile float*>(reinterpret_cast<uint8_t*>(bars) + 256);
  unsigned int* loss_warps = reinterpret_cast<unsigned int*>(reinterpret_cast<uint8_t*>(bars) + 272);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  const uint32_t acc_bar = bar_base + 8u * (2 * STAGES);
  const uint32_t recv_bar = bar_base + 8u * (2 * STAGES + 1);

  if (threadIdx.x == 0) {
    prefetch_tensormap(&map_a);       // descriptor fetch overlaps the rest of the prologue
    prefetch_tensormap(&map_b);
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(acc_bar, 1);
    mbar_init(recv_bar, 1);
    *abort_flag = 0;
    *loss_warps = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // this CTA will receive one column slice (BLOCK_N / split columns x 128 rows, fp32) from every peer
    mbar_arrive_expect_tx(recv_bar, (uint32_t)((split - 1) * (BLOCK_N / split) * BLOCK_M * 4));
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  cluster_arrive();                   // "my barriers are initialised"; the matching wait sits in front of the
  tc_fence_after();                   // first remote access (the slice exchange), off the main loop's path
  const uint32_t tmem_base = *tmem_slot;
  // tile and k-range of this CTA: index arithmetic only, done while the previous kernel drains
  const int tiles_m = (M + BLOCK_M - 1) / BLOCK_M;
  const int tile = blockIdx.x / split;
  const int m0 = (tile % tiles_m) * BLOCK_M, n0 = (tile / tiles_m) * BLOCK_N;
  const int num_k = (K + BLOCK_K - 1) / BLOCK_K;
  const int kpc = (num_k + split - 1) / split;
  const int kb_begin = min(num_k, (int)rank * kpc), kb_end = min(num_k, kb_begin + kpc);
  const int my_k = kb_end - kb_begin;     // may be 0 for the last ranks: they contribute zeros
  pdl_wait();
  pdl_trigger();

  // The k-loop of such a small product is bound by how fast one thread can issue the loads (a few hundred cycles
  // per k-block), so two threads share it: this warp announces the stage's bytes and loads the A tiles, the first
  // epilogue warp, idle until the accumulator is complete, loads the B tiles.  Both wait for the stage to be
  // free; bytes of B that land before the announcement only take the barrier's byte count below zero for a while
  // (the phase cannot complete before the announcing arrival).
  if (warp == 0) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        // the first pass over the ring finds every stage free: no wait (a wait that passes at once still costs a
        // couple of hundred cycles of the issuing thread)
        if (kb - kb_begin >= STAGES && !mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, dev_status)) break;
        mbar_arrive_expect_tx(full_bar(stage), (uint32_t)SPLITK_STAGE_BYTES);
        const uint32_t a_dst = smem_u32(smem_a + stage * A_TILE_BYTES);
        const int k0 = kb * BLOCK_K;
        if constexpr (A_MN) {
#pragma unroll
          for (int c = 0; c < BLOCK_M / CHUNK; ++c)
            tma_load_2d(a_dst + c * MN_CHUNK_BYTES, &map_a, m0 + c * CHUNK, k0, full_bar(stage));
        } else {
          tma_load_2d(a_dst, &map_a, k0, m0, full_bar(stage));
        }
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t fmt = TF32 ? 2u : 1u;
      constexpr uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((A_MN ? 1u : 0u) << 15) |
                                 ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(BLOCK_N >> 3) << 17) |
                                 ((uint32_t)(BLOCK_M >> 4) << 24);
      constexpr uint32_t a_lbo = A_MN ? MN_CHUNK_BYTES : 16, b_lbo = B_MN ? MN_CHUNK_BYTES : 16;
      constexpr uint32_t a_kstep = A_MN ? UMMA_K * TILE_ROW_BYTES : 32;
      constexpr uint32_t b_kstep = B_MN ? UMMA_K * TILE_ROW_BYTES : 32;
      constexpr uint32_t a_sbo = (TF32 && A_MN) ? 512 : 1024, b_sbo = (TF32 && B_MN) ? 512 : 1024;
      constexpr uint32_t a_lay = (TF32 && A_MN) ? 1 : 2, b_lay = (TF32 && B_MN) ? 1 : 2;
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int kb = 0; kb < my_k; ++kb) {
        if (!mbar_wait(full_bar(stage), phase, abort_flag, dev_status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t a_src = smem_u32(smem_a + stage * A_TILE_BYTES);
        const uint32_t b_src = smem_u32(smem_b + stage * B_TILE_BYTES);
#pragma unroll
        for (int kk = 0; kk < BLOCK_K / UMMA_K; ++kk) {
          const uint64_t da = make_smem_desc(a_src + kk * a_kstep, a_lbo, a_sbo, a_lay);
          const uint64_t db = make_smem_desc(b_src + kk * b_kstep, b_lbo, b_sbo, b_lay);
          tc_mma<TF32>(tmem_base, da, db, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
        }
        tc_commit(empty_bar(stage));
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
      if (ok) {
        if (my_k > 0) tc_commit(acc_bar);
        else mbar_arrive(acc_bar);          // nothing to contract: the epilogue treats the partial as zero
      }
    }
  } else {
    // ---------------- epilogue warps: reduce-scatter across the cluster, then the usual epilogue ------------
    if (warp == 2 && lane == 0) {                          // first: the B tiles of the main loop (see above)
      int stage = 0; uint32_t phase = 0;
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        // the first pass over the ring finds every stage free: no wait (a wait that passes at once still costs a
        // couple of hundred cycles of the issuing thread)
        if (kb - kb_begin >= STAGES && !mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, dev_status)) break;
        const uint32_t b_dst = smem_u32(smem_b + stage * B_TILE_BYTES);
        const int k0 = kb * BLOCK_K;
        if constexpr (B_MN) {
#pragma unroll
          for (int c = 0; c < BLOCK_N / CHUNK; ++c)
            tma_load_2d(b_dst + c * MN_CHUNK_BYTES, &map_b, n0 + c * CHUNK, k0, full_bar(stage));
        } else {
          tma_load_2d(b_dst, &map_b, k0, n0, full_bar(stage));
        }
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
    }
    __syncwarp();
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    const int row = m0 + row_in_tile;
    constexpr int w = W;                                   // columns owned by each CTA: 32, 16 or 8
    const int own_col0 = n0 + (int)rank * w;
    EpiSide side, tgt;                                     // side inputs of this CTA's slice, fetched ahead
    epilogue_prefetch<W>(epi, side, row, row < M, own_col0, min(N, own_col0 + w));
    if constexpr (LOSS) loss_prefetch_target<W>(epi.loss, tgt, row, row < M, own_col0, min(w, N - own_col0), N);
    float lacc = 0.f;
    bool ok = mbar_wait(acc_bar, 0, abort_flag, dev_status);
    tc_fence_after();
    const uint32_t slice_bytes = (uint32_t)(w * BLOCK_M * 4);
    float own[W];                                          // this CTA's slice of the tile
#pragma unroll
    for (int j = 0; j < W; ++j) own[j] = 0.f;
    if (ok) {
#pragma unroll 1
      for (int c = 0; c < BLOCK_N / 32; ++c) {
        float v[32];
        if (my_k > 0) {
          tmem_load_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * 32), v);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = 0.f;
        }
        // column c*32+j belongs to CTA (c*32+j)/w; the send buffer is [dest][col in slice][row], which is
        // simply [column][row]: consecutive lanes write consecutive floats
#pragma unroll
        for (int j = 0; j < 32; ++j) send[(c * 32 + j) * BLOCK_M + row_in_tile] = v[j];
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the bulk copies
      cluster_wait();                                                // every peer's receive barrier exists
      asm volatile("bar.sync 1, 128;" ::: "memory");                 // the four epilogue warps
      if (warp == 2 && lane == 0) {
        for (uint32_t dest = 0; dest < (uint32_t)split; ++dest) {
          if (dest == rank) continue;
          const uint32_t src = smem_u32(send + (int)dest * w * BLOCK_M);
          const uint32_t dst = map_to_cta(smem_u32(recv + (int)rank * w * BLOCK_M), dest);
          bulk_copy_to_peer(dst, src, slice_bytes, map_to_cta(recv_bar, dest));
        }
      }
      ok = mbar_wait(recv_bar, 0, abort_flag, dev_status);
    } else {
      cluster_wait();
    }
    if (ok) {
#pragma unroll
      for (int cs = 0; cs < W; ++cs) own[cs] = send[((int)rank * w + cs) * BLOCK_M + row_in_tile];
      for (int src = 0; src < split; ++src) {
        if ((uint32_t)src == rank) continue;
#pragma unroll
        for (int cs = 0; cs < W; ++cs) own[cs] += recv[(src * w + cs) * BLOCK_M + row_in_tile];
      }
      if (row < M && own_col0 < N) {
        if constexpr (LOSS) epilogue_store_mse(epi, own, side, tgt, row, own_col0, min(N, own_col0 + w), lacc);
        else epilogue_store(epi, own, side, row, own_col0, min(N, own_col0 + w));
      }
      if constexpr (LOSS) loss_finish(epi.loss, lacc, quarter, lane, loss_slots, loss_warps);
    }
    tc_fence_before();
  }

  __syncwarp();
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(20000);
  }
  if (warp < 2) cluster_wait();       // the producer and MMA warps complete the first cluster phase here
  tc_fence_before();
  __syncthreads();
  cluster_arrive();                   // no CTA leaves while a peer may still read its send buffer or write
  cluster_wait();                     // into its receive buffer
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
}


// ---- CTA-pair kernel (tcgen05 cta_group::2) ---------------------------------------------------------
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                                 uint32_t bar_cluster_addr) {
  // the completion barrier may live in the peer CTA of the pair
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// one arrival on the barrier at the same shared-memory offset in both CTAs of the pair, once all
// MMAs issued so far have completed
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
template <bool TF32>
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  if constexpr (TF32) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
  }
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

constexpr int PAIR_TILE_M = 256, PAIR_TILE_N = 256;
constexpr int PAIR_HALF_N = PAIR_TILE_N / 2;
constexpr int PAIR_B_BYTES = PAIR_HALF_N * TILE_ROW_BYTES;            // 16 KiB: this CTA's half of B
constexpr int PAIR_STAGE_BYTES = A_TILE_BYTES + PAIR_B_BYTES;         // 32 KiB per CTA per k-block
constexpr int PAIR_STAGES = 6;             // without output staging (the fused-update variant)
constexpr int PAIR_STAGES_STAGED = 5;      // with it: ring + staging stay within the same 192 KiB (measured: 4 stages +2 %, 3 stages +9 % step time)
constexpr int PAIR_SMEM = PAIR_STAGES * PAIR_STAGE_BYTES + SMEM_EXTRA;   // upper bound of both layouts

template <bool TF32, bool A_MN, bool B_MN, bool FUSED = false>
__global__ void __launch_bounds__(FUSED ? NUM_THREADS_FUSED : NUM_THREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    const __grid_constant__ CUtensorMap map_c, int M, int N, int K, EpilogueArgs epi, int* dev_status,
                    int group_m, int n_stages) {
  const int STAGES = n_stages;
  constexpr int BLOCK_K = TF32 ? 32 : 64;
  constexpr int UMMA_K = TF32 ? 8 : 16;
  constexpr int CHUNK = TF32 ? 32 : 64;
  constexpr int MN_CHUNK_BYTES = BLOCK_K * TILE_ROW_BYTES;
  constexpr uint32_t TMEM_COLS = 2 * PAIR_TILE_N;      // two 256-column accumulators per CTA

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + STAGES * A_TILE_BYTES;
  uint8_t* stage_out = smem + STAGES * PAIR_STAGE_BYTES;               // 1024-byte aligned
  uint64_t* bars = reinterpret_cast<uint64_t*>(stage_out + (epi.staged ? STAGE_OUT_BYTES : 0));
  // bars[0..S) full (used in the even CTA), [S..2S) empty, [2S..2S+2) tmem_full, [2S+2..2S+4) tmem_empty (even CTA)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  unsigned int* tiles_done = reinterpret_cast<unsigned int*>(tmem_slot + 2);   // FUSED: epilogue-warp arrivals

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();             // 0: issues the MMAs of the pair
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };

  if (threadIdx.x == 0) {
    prefetch_tensormap(&map_a);       // descriptor fetch overlaps the rest of the prologue
    prefetch_tensormap(&map_b);
    prefetch_tensormap(&map_c);
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }   // 4 warps x 2 CTAs
    *abort_flag = 0;
    *tiles_done = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  cluster_arrive();
  cluster_wait();                     // both CTAs' barriers exist before any cross-CTA signal
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // index arithmetic, the first tile's coordinates included: ahead of the dependency wait
  const int tiles_m = (M + PAIR_TILE_M - 1) / PAIR_TILE_M;
  const int tiles_n = (N + PAIR_TILE_N - 1) / PAIR_TILE_N;
  const int n_tiles = tiles_m * tiles_n;
  const int num_k = (K + BLOCK_K - 1) / BLOCK_K;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  int first_m = 0, first_n = 0;
  if (pair < n_tiles) tile_coords(pair, tiles_m, tiles_n, group_m, first_m, first_n);
  pdl_wait();
  pdl_trigger();

  if (warp == 0) {
    // ---------------- TMA producer (both CTAs; completion on the even CTA's barrier) ----------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int fills = 0;                     // as in the single-CTA kernel: no wait on the first pass over the ring
      bool ok = true;
      for (int t = pair; t < n_tiles && ok; t += n_pairs) {
        int m_idx, n_idx;
        if (t == pair) { m_idx = first_m; n_idx = first_n; } else tile_coords(t, tiles_m, tiles_n, group_m, m_idx, n_idx);
        const int m0 = m_idx * PAIR_TILE_M + (int)rank * BLOCK_M;
        const int n0 = n_idx * PAIR_TILE_N + (int)rank * PAIR_HALF_N;
        for (int kb = 0; kb < num_k; ++kb) {
          if (fills < STAGES) ++fills;
          else if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, dev_status)) { ok = false; break; }
          if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), (uint32_t)(2 * PAIR_STAGE_BYTES));
          const uint32_t fb = map_to_cta(full_bar(stage), 0);
          const uint32_t a_dst = smem_u32(smem_a + stage * A_TILE_BYTES);
          const uint32_t b_dst = smem_u32(smem_b + stage * PAIR_B_BYTES);
          const int k0 = kb * BLOCK_K;
          if constexpr (A_MN) {
#pragma unroll
            for (int c = 0; c < BLOCK_M / CHUNK; ++c)
              tma_load_2d_pair(a_dst + c * MN_CHUNK_BYTES, &map_a, m0 + c * CHUNK, k0, fb);
          } else {
            tma_load_2d_pair(a_dst, &map_a, k0, m0, fb);
          }
          if constexpr (B_MN) {
#pragma unroll
            for (int c = 0; c < PAIR_HALF_N / CHUNK; ++c)
              tma_load_2d_pair(b_dst + c * MN_CHUNK_BYTES, &map_b, n0 + c * CHUNK, k0, fb);
          } else {
            tma_load_2d_pair(b_dst, &map_b, k0, n0, fb);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: the even CTA only ----------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t fmt = TF32 ? 2u : 1u;
      constexpr uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((A_MN ? 1u : 0u) << 15) |
                                 ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(PAIR_TILE_N >> 3) << 17) |
                                 ((uint32_t)(PAIR_TILE_M >> 4) << 24);
      constexpr uint32_t a_lbo = A_MN ? MN_CHUNK_BYTES : 16, b_lbo = B_MN ? MN_CHUNK_BYTES : 16;
      constexpr uint32_t a_kstep = A_MN ? UMMA_K * TILE_ROW_BYTES : 32;
      constexpr uint32_t b_kstep = B_MN ? UMMA_K * TILE_ROW_BYTES : 32;
      constexpr uint32_t a_sbo = (TF32 && A_MN) ? 512 : 1024, b_sbo = (TF32 && B_MN) ? 512 : 1024;
      constexpr uint32_t a_lay = (TF32 && A_MN) ? 1 : 2, b_lay = (TF32 && B_MN) ? 1 : 2;
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      for (int t = pair; t < n_tiles && ok; t += n_pairs) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, dev_status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * PAIR_TILE_N);
        for (int kb = 0; kb < num_k; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, dev_status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = smem_u32(smem_a + stage * A_TILE_BYTES);
          const uint32_t b_src = smem_u32(smem_b + stage * PAIR_B_BYTES);
#pragma unroll
          for (int kk = 0; kk < BLOCK_K / UMMA_K; ++kk) {
            const uint64_t da = make_smem_desc(a_src + kk * a_kstep, a_lbo, a_sbo, a_lay);
            const uint64_t db = make_smem_desc(b_src + kk * b_kstep, b_lbo, b_sbo, b_lay);
            tc_mma_pair<TF32>(d_tmem, da, db, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          }
          tc_commit_pair(empty_bar(stage));       // frees this stage in both CTAs
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair(tfull_bar(acc));           // accumulator complete, both CTAs' epilogues may drain it
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp < NUM_THREADS / 32) {
    // ---------------- epilogue warps: each CTA drains its own 128 rows ----------------
    const int quarter = warp & 3;
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    for (int t = pair; t < n_tiles && ok; t += n_pairs) {
      int m_idx, n_idx;
      if (t == pair) { m_idx = first_m; n_idx = first_n; } else tile_coords(t, tiles_m, tiles_n, group_m, m_idx, n_idx);
      const int m0 = m_idx * PAIR_TILE_M + (int)rank * BLOCK_M;
      const int n0 = n_idx * PAIR_TILE_N;
      const int row = m0 + quarter * 32 + lane;
      EpiSide side, side_next;
      epilogue_prefetch(epi, side, row, row < M, n0, N);
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, dev_status)) { ok = false; break; }
      tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < PAIR_TILE_N / 32; ++c) {
        const int col0 = n0 + c * 32;
        if (col0 >= N) break;
        if (c + 1 < PAIR_TILE_N / 32) epilogue_prefetch(epi, side_next, row, row < M, col0 + 32, N);
        float v[32];
        tmem_load_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * PAIR_TILE_N + c * 32), v);
        if (FUSED || !epi.staged) {        // (the update warps read the tile back with ordinary loads: ordinary stores)
          if (row < M) epilogue_store(epi, v, side, row, col0, N);
        } else {
          epilogue_store_staged(epi, &map_c, stage_out + quarter * 2 * STAGE_OUT_WARP_BYTES, v, side, lane,
                                m0 + quarter * 32, col0, N, M, c);
        }
        side = side_next;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));
      if constexpr (FUSED) tile_stored_signal(tiles_done, lane);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) tma_store_wait_all();   // the staging buffers are read, and the output written, before the CTA leaves
  } else if constexpr (FUSED) {
    // ---------------- update warps: the optimizer on this CTA's 128 rows of every tile of the pair ----------------
    if (warp >= NUM_THREADS / 32) {
      const int uw = warp - NUM_THREADS / 32;
      float inv_bc1 = 1.0f, inv_bc2 = 1.0f;
      if (epi.upd.optimizer == SEG_ADAM) { inv_bc1 = 1.0f / __ldg(epi.upd.bc); inv_bc2 = 1.0f / __ldg(epi.upd.bc + 1); }
      unsigned int needed = 0;
      for (int t = pair; t < n_tiles; t += n_pairs) {
        needed += 4u;
        if (!tile_stored_wait(tiles_done, needed, abort_flag, dev_status, lane)) break;
        int m_idx, n_idx;
        if (t == pair) { m_idx = first_m; n_idx = first_n; } else tile_coords(t, tiles_m, tiles_n, group_m, m_idx, n_idx);
        const int m0 = m_idx * PAIR_TILE_M + (int)rank * BLOCK_M;
        const int n0 = n_idx * PAIR_TILE_N;
        update_tile<PAIR_TILE_N>(epi.upd, reinterpret_cast<const float*>(epi.C), epi.ldc, m0, n0, M, N, uw, lane,
                                 inv_bc1, inv_bc2);
      }
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(20000);
  }
  tc_fence_before();
  __syncthreads();
  cluster_arrive();                   // the pair releases its tensor memory together, after both are done
  cluster_wait();
  tc_fence_after();
  if (warp == 1) tmem_dealloc_pair(tmem_base, TMEM_COLS);
}

// ---- host side ---------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
constexpr int kMaxDevices = 64;

int current_device_slot() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
  return dev;
}
// SM count of the current device (cached per device; handles may live on different devices)
int num_sms() {
  static std::atomic<int> cache[kMaxDevices];
  const int slot = current_device_slot();
  int n = cache[slot].load(std::memory_order_relaxed);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, slot) != cudaSuccess || n <= 0) { cudaGetLastError(); return 148; }
  cache[slot].store(n, std::memory_order_relaxed);
  return n;
}
// cudaFuncSetAttribute once per kernel and device (the call itself is idempotent, so a race only repeats it)
template <typename Kern>
cudaError_t ensure_dynamic_smem(Kern kern, int bytes, std::atomic<bool>* flags) {
  std::atomic<bool>& done = flags[current_device_slot()];
  if (done.load(std::memory_order_acquire)) return cudaSuccess;
  cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (err == cudaSuccess) done.store(true, std::memory_order_release);
  return err;
}
std::once_flag g_init_once;
bool g_init_ok = false;
bool g_allow_splitk = true;
bool g_allow_pairs = true;
bool g_allow_fused_update = true;
bool g_staged_epilogue = true;      // SEG_NO_STAGED_EPILOGUE: per-lane stores instead of shared-memory staging + bulk stores
long g_pair_min_tiles = 0;      // SEG_PAIR_MIN_TILES: CTA pairs exactly from this many 256 x 256 tiles on (0: cost model)

// 2-D tensor map over a row-major matrix: `inner` contiguous elements per row, `outer` rows,
// `row_stride_bytes` between rows; box = box_inner x box_outer; 128-byte swizzle (32-byte atoms
// when atom32); zero fill.
bool make_map(CUtensorMap* map, bool f32, const void* base, uint64_t inner, uint64_t outer,
              uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_outer, bool atom32) {
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {row_stride_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                        const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Tensor map of the output C [M][N] (row pitch ldc) for the staged epilogue: boxes of 32 rows x 64 bytes (32 bf16 or
// 16 fp32 columns), 64-byte swizzle in shared memory.
bool make_output_map(CUtensorMap* map, bool f32, const void* base, uint64_t n_cols, uint64_t n_rows, uint64_t ldc) {
  cuuint64_t dims[2] = {n_cols, n_rows};
  cuuint64_t strides[1] = {ldc * (f32 ? 4u : 2u)};
  cuuint32_t box[2] = {f32 ? 16u : 32u, 32};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                        const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Rows of tiles per group of the tile order (see tile_coords): the largest group whose wave footprint - the operand
// panels of group_m row blocks plus those of the column blocks a wave of `ctas` tiles then spans - stays within a
// budget well under the L2 capacity; when even the squarest wave does not fit, the squarest wave.  Measured on the
// 8192 x 8192 x 4096 bf16 weight gradient: 354 MB of DRAM reads per launch against 735 MB in plain row-fastest order
// (operands 134 MB) and 4 % less time.  Where the squarest wave is still beyond the budget (K = 8192: 69 MB) the order
// changes nothing (610 MB either way), and L2 eviction-priority hints on the loads (row panels "evict last", column
// panels "evict first") raised the traffic instead (746-908 MB), as did nothing measurable for streaming stores of C.
constexpr long g_raster_budget_mb = 48;
int pick_group_m(int tiles_m, int tiles_n, int ctas, int tile_m, int tile_n, int K, int esz) {
  if ((long)tiles_m * tiles_n <= ctas) return tiles_m;            // one wave: nothing to keep
  const double row_mb = (double)tile_m * K * esz / 1048576.0, col_mb = (double)tile_n * K * esz / 1048576.0;
  for (int g = tiles_m; g >= 1; --g) {
    const int cols = std::min(tiles_n, (ctas + g - 1) / g);
    if (g * row_mb + cols * col_mb <= (double)g_raster_budget_mb) return g;
  }
  int best = 1;
  double best_mb = 1e30;
  for (int g = 1; g <= tiles_m; ++g) {
    const int cols = std::min(tiles_n, (ctas + g - 1) / g);
    const double mb = g * row_mb + cols * col_mb;
    if (mb < best_mb) { best_mb = mb; best = g; }
  }
  return best;
}

template <bool TF32, bool A_MN, bool B_MN, int BLOCK_N, bool FUSED = false>
cudaError_t launch_variant(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const GemmDesc& g,
                           const EpilogueArgs& e, int* dev_status, cudaStream_t s) {
  using L = SmemLayout<BLOCK_N>;
  auto kern = gemm_tc_kernel<TF32, A_MN, B_MN, BLOCK_N, FUSED>;
  static std::atomic<bool> attr_set_dev[kMaxDevices];      // the attribute is per device
  if (cudaError_t err = ensure_dynamic_smem(kern, L::TOTAL, attr_set_dev); err != cudaSuccess) return err;
  const int tiles = ((g.M + BLOCK_M - 1) / BLOCK_M) * ((g.N + BLOCK_N - 1) / BLOCK_N);
  const int grid = tiles < num_sms() ? tiles : num_sms();
  const int group_m = pick_group_m((g.M + BLOCK_M - 1) / BLOCK_M, (g.N + BLOCK_N - 1) / BLOCK_N, grid, BLOCK_M, BLOCK_N, g.K,
                                   TF32 ? 4 : 2);
  const int n_stages = e.staged ? L::STAGES_STAGED : L::STAGES;
  const int smem_bytes = n_stages * L::STAGE_BYTES + (e.staged ? STAGE_OUT_BYTES : 0) + SMEM_EXTRA;
  return launch_k(kern, dim3(grid), dim3(FUSED ? NUM_THREADS_FUSED : NUM_THREADS), smem_bytes, s, ma, mb, mc, g.M, g.N, g.K,
                  e, dev_status, group_m, n_stages);
}

template <bool TF32, int BLOCK_N>
cudaError_t launch_majors(bool a_mn, bool b_mn, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc,
                          const GemmDesc& g, const EpilogueArgs& e, int* dev_status, cudaStream_t s) {
  if (!a_mn && !b_mn) return launch_variant<TF32, false, false, BLOCK_N>(ma, mb, mc, g, e, dev_status, s);
  if (!a_mn && b_mn) return launch_variant<TF32, false, true, BLOCK_N>(ma, mb, mc, g, e, dev_status, s);
  if (a_mn && b_mn) {
    if (e.upd.enabled) return launch_variant<TF32, true, true, BLOCK_N, true>(ma, mb, mc, g, e, dev_status, s);
    return launch_variant<TF32, true, true, BLOCK_N>(ma, mb, mc, g, e, dev_status, s);
  }
  return cudaErrorNotSupported;
}


template <bool TF32, bool A_MN, bool B_MN, int SPLIT, bool LOSS = false>
cudaError_t launch_splitk_cluster(const CUtensorMap& ma, const CUtensorMap& mb, const GemmDesc& g,
                                  const EpilogueArgs& e, int* dev_status, cudaStream_t s) {
  constexpr int split = SPLIT;
  auto kern = gemm_tc_splitk_kernel<TF32, A_MN, B_MN, SPLIT, LOSS>;
  static std::atomic<bool> attr_set_dev[kMaxDevices];      // the attribute is per device
  if (cudaError_t err = ensure_dynamic_smem(kern, SPLITK_SMEM, attr_set_dev); err != cudaSuccess) return err;
  const int tiles = ((g.M + BLOCK_M - 1) / BLOCK_M) * ((g.N + SPLITK_BLOCK_N - 1) / SPLITK_BLOCK_N);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(tiles * split), 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = SPLITK_SMEM;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)split; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = g_use_pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kern, ma, mb, g.M, g.N, g.K, e, dev_status);
}

template <bool TF32, bool A_MN, bool B_MN, bool LOSS = false>
cudaError_t launch_splitk_variant(const CUtensorMap& ma, const CUtensorMap& mb, const GemmDesc& g,
                                  const EpilogueArgs& e, int split, int* dev_status, cudaStream_t s) {
  switch (split) {
    case 2: return launch_splitk_cluster<TF32, A_MN, B_MN, 2, LOSS>(ma, mb, g, e, dev_status, s);
    case 4: return launch_splitk_cluster<TF32, A_MN, B_MN, 4, LOSS>(ma, mb, g, e, dev_status, s);
    default: return cudaErrorNotSupported;                  // pick_split chooses 2 or 4
  }
}

template <bool TF32>
cudaError_t launch_splitk_majors(bool a_mn, bool b_mn, const CUtensorMap& ma, const CUtensorMap& mb,
                                 const GemmDesc& g, const EpilogueArgs& e, int split, int* dev_status, cudaStream_t s) {
  if (!a_mn && !b_mn) {
    if (e.loss.enabled) return launch_splitk_variant<TF32, false, false, true>(ma, mb, g, e, split, dev_status, s);
    return launch_splitk_variant<TF32, false, false>(ma, mb, g, e, split, dev_status, s);
  }
  if (!a_mn && b_mn) return launch_splitk_variant<TF32, false, true>(ma, mb, g, e, split, dev_status, s);
  if (a_mn && b_mn) return launch_splitk_variant<TF32, true, true>(ma, mb, g, e, split, dev_status, s);
  return cudaErrorNotSupported;
}

// Split K over a cluster when the 128 x 64 tiles alone would leave most SMs idle and K is long
// enough that the main loop, not the fixed cost, dominates.  Returns 1 for "do not split".
int pick_split(int M, int N, int K, bool tf32) {
  const int tiles = ((M + BLOCK_M - 1) / BLOCK_M) * ((N + SPLITK_BLOCK_N - 1) / SPLITK_BLOCK_N);
  const int num_k = (K + (tf32 ? 32 : 64) - 1) / (tf32 ? 32 : 64);
  // measured: a k-block costs about 0.27 us of one SM's shared-memory fill time, the cluster exchange about 2 us
  int best = 1;
  double best_us = 0.27 * num_k;
  for (int sp : {2, 4}) {
    if (tiles * sp > num_sms()) break;
    const double us = 0.27 * ((num_k + sp - 1) / sp) + 2.0;
    if (us < best_us - 0.5) { best = sp; best_us = us; }
  }
  return best;
}

template <bool TF32, bool A_MN, bool B_MN, bool FUSED = false>
cudaError_t launch_pair_variant(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const GemmDesc& g,
                                const EpilogueArgs& e, int* dev_status, cudaStream_t s) {
  auto kern = gemm_tc_pair_kernel<TF32, A_MN, B_MN, FUSED>;
  static std::atomic<bool> attr_set_dev[kMaxDevices];      // the attribute is per device
  if (cudaError_t err = ensure_dynamic_smem(kern, PAIR_SMEM, attr_set_dev); err != cudaSuccess) return err;
  const int tiles = ((g.M + PAIR_TILE_M - 1) / PAIR_TILE_M) * ((g.N + PAIR_TILE_N - 1) / PAIR_TILE_N);
  const int pairs = std::min(tiles, num_sms() / 2);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
  cfg.blockDim = dim3(FUSED ? NUM_THREADS_FUSED : NUM_THREADS, 1, 1);
  const int n_stages = e.staged ? PAIR_STAGES_STAGED : PAIR_STAGES;
  cfg.dynamicSmemBytes = n_stages * PAIR_STAGE_BYTES + (e.staged ? STAGE_OUT_BYTES : 0) + SMEM_EXTRA;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = g_use_pdl ? 2 : 1;
  const int group_m = pick_group_m((g.M + PAIR_TILE_M - 1) / PAIR_TILE_M, (g.N + PAIR_TILE_N - 1) / PAIR_TILE_N, pairs,
                                   PAIR_TILE_M, PAIR_TILE_N, g.K, TF32 ? 4 : 2);
  return cudaLaunchKernelEx(&cfg, kern, ma, mb, mc, g.M, g.N, g.K, e, dev_status, group_m, n_stages);
}

template <bool TF32>
cudaError_t launch_pair_majors(bool a_mn, bool b_mn, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc,
                               const GemmDesc& g, const EpilogueArgs& e, int* dev_status, cudaStream_t s) {
  if (!a_mn && !b_mn) return launch_pair_variant<TF32, false, false>(ma, mb, mc, g, e, dev_status, s);
  if (!a_mn && b_mn) return launch_pair_variant<TF32, false, true>(ma, mb, mc, g, e, dev_status, s);
  if (a_mn && b_mn) {
    if (e.upd.enabled) return launch_pair_variant<TF32, true, true, true>(ma, mb, mc, g, e, dev_status, s);
    return launch_pair_variant<TF32, true, true>(ma, mb, mc, g, e, dev_status, s);
  }
  return cudaErrorNotSupported;
}

// Kernel selection by a cost model of the main loop.  One CTA's main loop is bound by the rate at
// which one SM's shared memory is filled (about 64 bytes per clock, measured: 24 KiB of operands per
// k-block take 0.2 us, 32 KiB 0.27 us, 48 KiB 0.4 us); a CTA pair stages 32 KiB per CTA for the work
// a single CTA needs 48 KiB for.  Persistent kernels run ceil(tiles / CTAs) rounds of num_k k-blocks.
struct Choice { int kind; int block_n; double us; };      // kind 0: single CTA, 1: CTA pair
Choice pick_kernel(int M, int N, int K, bool tf32, bool throughput) {
  const int num_k = (K + (tf32 ? 32 : 64) - 1) / (tf32 ? 32 : 64);
  const int tiles_m = (M + BLOCK_M - 1) / BLOCK_M;
  Choice best{0, 64, 1e30};
  for (int bn : {64, 128, 256}) {
    if (bn > 64 && bn / 2 >= N) continue;                  // do not use a tile twice as wide as N
    const long tiles = (long)tiles_m * ((N + bn - 1) / bn);
    const long rounds = (tiles + num_sms() - 1) / num_sms();
    const double per_kb = (16.0 + bn / 8.0) / 120.0;       // KiB per k-block / (KiB per us)
    double us = rounds * (num_k * per_kb + 0.4 + bn / 128.0);   // + per-tile epilogue not hidden
    // beside other kernels the SM time taken counts as well: latency + tiles x time of a tile / SMs, with the
    // measured fixed cost of a tile (wider tiles drain more columns and allocate more tensor memory)
    if (throughput) {
      const double t = num_k * per_kb + 3.5 + bn / 48.0;
      us = rounds * t + (double)tiles * t / num_sms();
    }
    if (us < best.us) best = Choice{0, bn, us};
  }
  if (g_allow_pairs && M >= 256 && N >= 256 && K >= 256) {
    const long tiles = (long)((M + PAIR_TILE_M - 1) / PAIR_TILE_M) * ((N + PAIR_TILE_N - 1) / PAIR_TILE_N);
    const long pairs = num_sms() / 2;
    const long rounds = (tiles + pairs - 1) / pairs;
    double us = rounds * (num_k * (32.0 / 120.0) + 0.4 + 2.0);
    if (throughput) {
      const double t = num_k * (32.0 / 120.0) + 9.0;          // measured: a pair's fixed cost is about 9 us
      us = rounds * t + (double)(2 * tiles) * t / num_sms();
    }
    if (g_pair_min_tiles > 0) {                            // diagnostic override: pairs from that many tiles on
      if (tiles >= g_pair_min_tiles) best = Choice{1, PAIR_HALF_N, us};
    } else if (us < best.us) {
      best = Choice{1, PAIR_HALF_N, us};
    }
  }
  return best;
}

}  // namespace

bool gemm_tc_init() {
  std::call_once(g_init_once, [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || fn == nullptr) {
      cudaGetLastError();
      return;
    }
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    const char* env = getenv("SEG_NO_SPLITK");
    if (env && env[0] == '1') g_allow_splitk = false;
    env = getenv("SEG_NO_PAIRS");
    if (env && env[0] == '1') g_allow_pairs = false;
    env = getenv("SEG_PAIR_MIN_TILES");
    if (env) g_pair_min_tiles = atol(env);
    env = getenv("SEG_NO_STAGED_EPILOGUE");
    if (env && env[0] == '1') g_staged_epilogue = false;
    g_init_ok = true;
  });
  return g_init_ok;
}

// ---- self-test of the bounded wait ---------------------------------------------------------------
namespace {
__global__ void __launch_bounds__(32)
wait_selftest_kernel(int* dev_status, uint64_t limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // nothing ever arrives at this barrier: the wait below ends only through its own time limit
    mbar_wait(smem_u32(&bar), 0, &abort_flag, dev_status, limit_ns);
  }
}
}  // namespace

cudaError_t launch_wait_selftest(int* dev_status, uint64_t limit_ns, cudaStream_t s) {
  wait_selftest_kernel<<<1, 32, 0, s>>>(dev_status, limit_ns);
  return cudaGetLastError();
}

// The mean-squared-error loss of a non-final segment is fused into the split-K kernel, the one that
// serves the small, latency-bound products: there it replaces a launch on the critical path for about
// 3 us of extra epilogue (paper_shaped: -3 us per step).  In the single-CTA kernel of mid-sized
// products the same epilogue measured slower than the separate loss launch (bf16_wide 1024x2048x4096:
// 44 us against 25 + 14 us under ncu), and the CTA-pair kernel serves large products, where a separate
// loss launch costs next to nothing.  Softmax cross-entropy was tried in the epilogue of the single-CTA
// kernel in three forms - one thread per row of at most 64 logits unrolled in registers (3-4 times slower
// than the separate warp-per-row kernel), the tile left in shared memory with each warp walking its 32
// rows, lanes over the classes (slower still: 32 dependent reduction chains per warp), and one thread
// per row with short loops over its row in shared memory (about the cost of the launch it saves, and
// it gives up the split over K) - and stays a launch of its own.
bool gemm_tc_can_fuse_loss(int M, int N, int K, bool tf32) {
  if (!g_init_ok || !g_allow_splitk) return false;
  return pick_split(M, N, K, tf32) > 1;
}

// The fused update lives in the persistent kernels (one CTA or a CTA pair per tile); products small enough to
// be split over K keep the separate update launch, and so does anything the tensor-core path cannot take.
bool gemm_tc_can_fuse_update(const GemmDesc& g) {
  if (!g_init_ok || !g_allow_fused_update) return false;
  if (g.epi != EPI_PLAIN || g.a_sm != 1 || g.b_sn != 1 || g.c_dt != DT_F32 || g.a_dt != g.b_dt) return false;
  if (g.M <= 0 || g.N <= 0 || g.K <= 0) return false;
  const bool tf32 = (g.a_dt == DT_F32);
  const int esz = tf32 ? 4 : 2;
  if ((reinterpret_cast<uintptr_t>(g.A) & 15u) || (reinterpret_cast<uintptr_t>(g.B) & 15u)) return false;
  if ((g.a_sk * esz) % 16 != 0 || (g.b_sk * esz) % 16 != 0) return false;
  if ((reinterpret_cast<uintptr_t>(g.C) & 15u) || (g.ldc & 3)) return false;
  const bool throughput = g.off_critical_path != 0;
  const int split = (g_allow_splitk && !throughput) ? pick_split(g.M, g.N, g.K, tf32) : 1;
  return split == 1;
}

cudaError_t launch_gemm_tc(const GemmDesc& g, int* dev_status, cudaStream_t s, int* family) {
  if (!g_init_ok) return cudaErrorNotSupported;
  if (g.M <= 0 || g.N <= 0 || g.K <= 0) return cudaErrorNotSupported;
  if (g.a_dt != g.b_dt) return cudaErrorNotSupported;
  const bool tf32 = (g.a_dt == DT_F32);
  const int esz = tf32 ? 4 : 2;
  // operand majors from the strides
  bool a_mn, b_mn;
  int64_t a_pitch, b_pitch;
  if (g.a_sk == 1) { a_mn = false; a_pitch = g.a_sm; }
  else if (g.a_sm == 1) { a_mn = true; a_pitch = g.a_sk; }
  else return cudaErrorNotSupported;
  if (g.b_sk == 1) { b_mn = false; b_pitch = g.b_sn; }
  else if (g.b_sn == 1) { b_mn = true; b_pitch = g.b_sk; }
  else return cudaErrorNotSupported;
  if (a_mn && !b_mn) return cudaErrorNotSupported;
  // TMA rules: 16-byte aligned base, row pitch a multiple of 16 bytes
  if ((reinterpret_cast<uintptr_t>(g.A) & 15u) || (reinterpret_cast<uintptr_t>(g.B) & 15u)) return cudaErrorNotSupported;
  if ((a_pitch * esz) % 16 != 0 || (b_pitch * esz) % 16 != 0) return cudaErrorNotSupported;
  if (a_pitch * (int64_t)esz >= (1ll << 40) || b_pitch * (int64_t)esz >= (1ll << 40)) return cudaErrorNotSupported;

  const bool fuse_loss = (g.epi == EPI_BIAS_ACT) && g.loss.enabled != 0;
  if (fuse_loss && (a_mn || b_mn || !gemm_tc_can_fuse_loss(g.M, g.N, g.K, tf32)))
    return cudaErrorInvalidValue;                           // the caller asks gemm_tc_can_fuse_loss first
  const bool throughput = g.off_critical_path != 0;
  const int split = (g_allow_splitk && !throughput) ? pick_split(g.M, g.N, g.K, tf32) : 1;
  const Choice choice = pick_kernel(g.M, g.N, g.K, tf32, throughput);
  const bool pairs = (split == 1) && choice.kind == 1;
  const int block_n = split > 1 ? SPLITK_BLOCK_N : choice.block_n;
  const uint32_t block_k = tf32 ? 32 : 64, chunk = tf32 ? 32 : 64;
  CUtensorMap ma, mb;
  bool ok;
  if (!a_mn) ok = make_map(&ma, tf32, g.A, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)a_pitch * esz, block_k, BLOCK_M, false);
  else ok = make_map(&ma, tf32, g.A, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)a_pitch * esz, chunk, block_k, tf32);
  if (!ok) return cudaErrorNotSupported;
  if (!b_mn) ok = make_map(&mb, tf32, g.B, (uint64_t)g.K, (uint64_t)g.N, (uint64_t)b_pitch * esz, block_k, (uint32_t)block_n, false);
  else ok = make_map(&mb, tf32, g.B, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)b_pitch * esz, chunk, block_k, tf32);
  if (!ok) return cudaErrorNotSupported;

  EpilogueArgs e;
  e.C = g.C; e.ldc = g.ldc; e.c_dt = g.c_dt; e.c_round = g.c_round; e.epi = g.epi; e.relu = g.relu;
  e.bias = g.bias; e.mask = g.mask; e.ldmask = g.ldmask;
  e.loss = g.loss; e.loss.enabled = fuse_loss ? 1 : 0;
  e.upd = g.upd;
  e.staged = (g_staged_epilogue && !e.upd.enabled) ? 1 : 0;
  if (e.upd.enabled && (split > 1 || !a_mn || !b_mn || g.epi != EPI_PLAIN || g.c_dt != DT_F32))
    return cudaErrorInvalidValue;                           // the caller asks gemm_tc_can_fuse_update first

  // output map of the persistent kernels' staged epilogue (the split-K kernel stores its column slices itself)
  CUtensorMap mc;
  if (split == 1) {
    if ((reinterpret_cast<uintptr_t>(g.C) & 15u) || (g.ldc * (g.c_dt == DT_F32 ? 4 : 2)) % 16 != 0) return cudaErrorNotSupported;
    if (!make_output_map(&mc, g.c_dt == DT_F32, g.C, (uint64_t)g.N, (uint64_t)g.M, (uint64_t)g.ldc)) return cudaErrorNotSupported;
  }
  if (family) *family = pairs ? FAM_TC_PAIR : (split > 1 ? FAM_TC_SPLITK : FAM_TC_SINGLE);
  if (pairs) {
    return tf32 ? launch_pair_majors<true>(a_mn, b_mn, ma, mb, mc, g, e, dev_status, s)
                : launch_pair_majors<false>(a_mn, b_mn, ma, mb, mc, g, e, dev_status, s);
  }
  if (split > 1) {
    return tf32 ? launch_splitk_majors<true>(a_mn, b_mn, ma, mb, g, e, split, dev_status, s)
                : launch_splitk_majors<false>(a_mn, b_mn, ma, mb, g, e, split, dev_status, s);
  }
#define SEGK_TC(TF, BN) launch_majors<TF, BN>(a_mn, b_mn, ma, mb, mc, g, e, dev_status, s)
  if (tf32) {
    if (block_n == 256) return SEGK_TC(true, 256);
    if (block_n == 128) return SEGK_TC(true, 128);
    return SEGK_TC(true, 64);
  }
  if (block_n == 256) return SEGK_TC(false, 256);
  if (block_n == 128) return SEGK_TC(false, 128);
  return SEGK_TC(false, 64);
#undef SEGK_TC
}

}  // namespace segk
