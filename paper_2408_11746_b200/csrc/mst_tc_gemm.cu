// bf16 contraction on the 5th-generation tensor cores (tcgen05) with fp32 accumulators in tensor memory.
//
// One persistent block per SM, 192 threads in three roles:
//   warp 0     producer: one lane issues TMA tile loads (cp.async.bulk.tensor, 128-byte swizzle) into a 4-stage
//              shared-memory ring, signalling "full" mbarriers by transaction bytes;
//   warp 1     one lane issues tcgen05.mma (M=128, N=256, K=16 per instruction) from shared-memory descriptors
//              into one of two 128x256 fp32 accumulators in tensor memory, tcgen05.commit releases the smem stage
//              ("empty") and, after the last K block, hands the accumulator to the epilogue ("tmem_full");
//   warps 2-9  epilogue, two warps per tensor-memory lane quarter taking alternate 32-column chunks: tcgen05.ld
//              (one row per thread), convert / activate / sample / store, then release the accumulator
//              ("tmem_empty") so the next tile's MMAs overlap this tile's stores.
// Operands may be K-major ([rows x K] row-major) or MN-major ([K x rows] row-major, as dY and X are for
// G = dY^T X): the tile is fetched with 64-element-wide boxes either way and described to the tensor core with the
// matching canonical layout (K-major: 8-row groups 1024 B apart; MN-major: 64-wide blocks one box apart).
// Every mbarrier wait is bounded: on expiry the block raises an abort flag, records an error bit, skips the rest
// of its work, frees its tensor memory and returns.
#include "mst_tc_gemm.cuh"

#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdlib>

#include "mst_internal.cuh"
#include "mst_tc_ptx.cuh"

namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2;  // 16 KiB
constexpr int B_BYTES = BN * BK * 2;  // 32 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int BOX_BYTES = 64 * BK * 2;  // one 64-wide MN-major box: 8 KiB
constexpr int EPI_WARPS = 8;  // two per tensor-memory lane quarter, alternating 32-column chunks
constexpr int NUM_THREADS = 64 + 32 * EPI_WARPS;
constexpr int TMEM_COLS = 512;
constexpr int OUT_BOX_BYTES = 32 * 128;  // one epilogue warp's staging box: 32 rows x 128 bytes
constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + EPI_WARPS * OUT_BOX_BYTES + 1024 /*align*/ + 256 /*barriers*/;

__device__ int g_tc_error = 0;  // sticky: 1 = a bounded wait expired

struct Params {
  int64_t M, N;
  int kblocks;        // ceil(K / BK)
  int splits;
  int m_tiles, n_tiles;
  int a_mn, b_mn;
  int epilogue;
  void* out;
  int64_t ldc;
  float* partial;
  const uint32_t* bits;
  const int32_t* wscan;
  int wpr;
  int64_t nnz;
  int act;
  void* pre;
  int64_t ldpre;
  int tma_out;  // rows leave through shared memory and TMA stores (tensor map tmC) instead of per-thread stores
  int sampled_stage_min;  // sampled output: a 32 x 32 chunk with at least this many kept entries leaves row by row
};

// PTX wrappers live in mst_tc_ptx.cuh; waits in this file report to g_tc_error
using namespace mst_ptx;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return mst_ptx::mbar_wait(bar, parity, abort_flag, &g_tc_error);
}

// Phi(x) and exp(-x^2/2) for the fused activation.  The complementary error function is the five-term rational
// approximation of Abramowitz & Stegun 7.1.26 (absolute error below 1.5e-7, far under the bf16 rounding of the
// result); it shares its exponential with the normal density, and Phi of a negative argument is formed without
// cancellation.  It costs about a third of erff's instructions (flush-to-zero reciprocal and exp2, whose default
// forms carry denormal handling); the epilogue is still the slower side of the overlap when an activation is fused.
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void phi_fast(float x, float& cdf, float& e) {
  const float z = fabsf(x) * 0.70710678118654752f;
  const float t = rcp_approx(fmaf(0.3275911f, z, 1.0f));
  e = ex2_approx(x * x * -0.72134752044448170f);  // exp(-x^2 / 2)
  float poly = fmaf(t, 1.061405429f, -1.453152027f);
  poly = fmaf(poly, t, 1.421413741f);
  poly = fmaf(poly, t, -0.284496736f);
  poly = fmaf(poly, t, 0.254829592f);
  const float q = 0.5f * poly * t * e;  // Phi(-|x|)
  cdf = x >= 0.0f ? 1.0f - q : q;
}
__device__ __forceinline__ float gelu_fast(float x) {
  float cdf, e;
  phi_fast(x, cdf, e);
  return x * cdf;
}
__device__ __forceinline__ float gelu_grad_fast(float x) {
  float cdf, e;
  phi_fast(x, cdf, e);
  return fmaf(x * 0.39894228040143268f, e, cdf);
}

// Activation step of one 32-column chunk held in registers (row m, columns n..n+31).  GELU: r <- gelu(r), the
// pre-activation going to P.pre when given; GELU_GRAD: r <- r * gelu'(pre), pre already fetched into p4 when pre_vec.
__device__ __forceinline__ void act_chunk(const Params& P, uint32_t (&r)[32], uint16_t* pre, bool pre_vec, const uint4 (&p4)[4],
                                          int n) {
  if (P.act == MST_ACT_GELU) {
    if (P.pre) {  // keep the pre-activation for the backward pass
      if (pre_vec) {
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint4 o;
          o.x = pack_bf16(__uint_as_float(r[8 * v + 0]), __uint_as_float(r[8 * v + 1]));
          o.y = pack_bf16(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3]));
          o.z = pack_bf16(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5]));
          o.w = pack_bf16(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7]));
          reinterpret_cast<uint4*>(pre)[v] = o;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (n + j < P.N) pre[j] = (uint16_t)(pack_bf16(__uint_as_float(r[j]), 0.f) & 0xFFFFu);
      }
    }
#pragma unroll
    for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(gelu_fast(__uint_as_float(r[j])));
  } else {  // multiply by the derivative at the stored pre-activation
    if (pre_vec) {
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        const uint32_t pw[4] = {p4[v].x, p4[v].y, p4[v].z, p4[v].w};
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          const float lo = __uint_as_float(pw[h] << 16), hi = __uint_as_float(pw[h] & 0xFFFF0000u);
          r[8 * v + 2 * h] = __float_as_uint(__uint_as_float(r[8 * v + 2 * h]) * gelu_grad_fast(lo));
          r[8 * v + 2 * h + 1] = __float_as_uint(__uint_as_float(r[8 * v + 2 * h + 1]) * gelu_grad_fast(hi));
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (n + j < P.N)
          r[j] = __float_as_uint(__uint_as_float(r[j]) * gelu_grad_fast(__uint_as_float((uint32_t)pre[j] << 16)));
    }
  }
}

// One 128 x BN accumulator (tensor-memory lanes = rows) -> global memory, 32 columns at a time, each thread storing
// its own row.  q = lane quarter this warp may read, m0/n0 = first row / column of this block's tile.
// c0 = first chunk this warp takes; the warps of one lane quarter interleave their chunks.
__device__ __forceinline__ void epilogue_tile(const Params& P, uint32_t tmem_base, int acc, int q, int c0, int lane,
                                              int64_t m0, int n0, int split) {
  const int64_t m = (int64_t)m0 + q * 32 + lane;
  const bool row_ok = m < P.M;
#pragma unroll 1
  for (int c = c0; c < BN / 32; c += EPI_WARPS / 4) {
    const int n = n0 + c * 32;
    if (n >= P.N) break;  // uniform
    uint32_t r[32];
    // derivative mode: the stored pre-activation of this chunk is fetched ahead of the tensor-memory read
    uint16_t* pre = reinterpret_cast<uint16_t*>(P.pre) + m * P.ldpre + n;
    const bool pre_vec = n + 32 <= P.N && ((P.ldpre & 7) == 0) && ((reinterpret_cast<uintptr_t>(P.pre) & 15u) == 0);
    uint4 p4[4];
    if (P.act == MST_ACT_GELU_GRAD && pre_vec && row_ok) {
#pragma unroll
      for (int v = 0; v < 4; ++v) p4[v] = __ldg(reinterpret_cast<const uint4*>(pre) + v);
    }
    tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + c * 32), r);
    if (!row_ok) continue;
    if (P.epilogue == MST_TC_OUT_BF16) {
      if (P.act) act_chunk(P, r, pre, pre_vec, p4, n);
      uint16_t* dst = reinterpret_cast<uint16_t*>(P.out) + m * P.ldc + n;
      if (n + 32 <= P.N && ((P.ldc & 7) == 0) && ((reinterpret_cast<uintptr_t>(P.out) & 15u) == 0)) {
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint4 o;
          o.x = pack_bf16(__uint_as_float(r[8 * v + 0]), __uint_as_float(r[8 * v + 1]));
          o.y = pack_bf16(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3]));
          o.z = pack_bf16(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5]));
          o.w = pack_bf16(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7]));
          reinterpret_cast<uint4*>(dst)[v] = o;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (n + j < P.N) dst[j] = (uint16_t)(pack_bf16(__uint_as_float(r[j]), 0.f) & 0xFFFFu);
      }
    } else if (P.epilogue == MST_TC_OUT_F32) {
      float* base = P.splits > 1 ? P.partial + (int64_t)split * P.M * P.N + m * P.N : reinterpret_cast<float*>(P.out) + m * P.ldc;
      float* dst = base + n;
      const int64_t ld = P.splits > 1 ? P.N : P.ldc;
      if (n + 32 <= P.N && ((ld & 3) == 0) && ((reinterpret_cast<uintptr_t>(base) & 15u) == 0)) {
#pragma unroll
        for (int v = 0; v < 8; ++v)
          reinterpret_cast<uint4*>(dst)[v] = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (n + j < P.N) dst[j] = __uint_as_float(r[j]);
      }
    } else {
      // sampled: the 32 columns of this chunk are one mask word of row m
      const int64_t wi = m * P.wpr + (n >> 5);
      const uint32_t word = P.bits[wi];
      float* dst = (P.splits > 1 ? P.partial + (int64_t)split * P.nnz : reinterpret_cast<float*>(P.out)) + P.wscan[wi];
      if (word == 0xFFFFFFFFu) {
        // dense stretch (a restored layer, a saturated row): the 32 values are contiguous in CSR order
#pragma unroll
        for (int j = 0; j < 32; ++j) dst[j] = __uint_as_float(r[j]);
      } else {
        int rank = 0;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          if ((word >> j) & 1u) {
            dst[rank] = __uint_as_float(r[j]);
            ++rank;
          }
        }
      }
    }
  }
}

// The sampled accumulator (weight gradient under the mask).  A chunk is 32 rows x one mask word.  Chunks with few
// entries are written by the row-owning lanes, entry by entry.  Denser chunks leave through the warp's staging box:
// the lanes turn from rows to columns, so that each store instruction writes the kept entries of ONE row, which are
// neighbours in CSR order; a row-per-lane store touches 32 lines per instruction and costs the memory pipeline as many
// passes, which at high density slows the concurrent main loop.
__device__ __forceinline__ void epilogue_tile_sampled(const Params& P, uint32_t stage, uint32_t tmem_base, int acc, int q,
                                                      int c0, int lane, int64_t m0, int n0, int split) {
  const int64_t m = (int64_t)m0 + q * 32 + lane;
  const bool row_ok = m < P.M;
  const uint32_t my_row = stage + (uint32_t)lane * 128u;
  const uint32_t sw = (uint32_t)(lane & 7);
  const uint32_t lt = (1u << lane) - 1u;
  float* out = P.splits > 1 ? P.partial + (int64_t)split * P.nnz : reinterpret_cast<float*>(P.out);
#pragma unroll 1
  for (int c = c0; c < BN / 32; c += EPI_WARPS / 4) {
    const int n = n0 + c * 32;
    if (n >= P.N) break;  // uniform
    uint32_t word = 0;
    int32_t at = 0;
    if (row_ok) {
      const int64_t wi = m * P.wpr + (n >> 5);
      word = P.bits[wi];
      at = P.wscan[wi];
    }
    uint32_t r[32];
    tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + c * 32), r);
    const int kept = __reduce_add_sync(0xFFFFFFFFu, __popc(word));
    if (kept < P.sampled_stage_min) {
      float* dst = out + at;
      int rank = 0;
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        if ((word >> j) & 1u) {
          dst[rank] = __uint_as_float(r[j]);
          ++rank;
        }
      }
      continue;
    }
    __syncwarp();  // the previous chunk has been read out of the box
#pragma unroll
    for (int v = 0; v < 8; ++v) {
      const uint32_t piece = (uint32_t)v ^ sw;
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(my_row + piece * 16u), "r"(r[4 * v]), "r"(r[4 * v + 1]),
                   "r"(r[4 * v + 2]), "r"(r[4 * v + 3])
                   : "memory");
    }
    __syncwarp();
#pragma unroll 4
    for (int rr = 0; rr < 32; ++rr) {
      const uint32_t w = __shfl_sync(0xFFFFFFFFu, word, rr);
      const int32_t base = __shfl_sync(0xFFFFFFFFu, at, rr);
      if (w == 0) continue;  // uniform
      const uint32_t piece = (uint32_t)(lane >> 2) ^ (uint32_t)(rr & 7);
      uint32_t v;
      asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(stage + (uint32_t)rr * 128u + piece * 16u + (uint32_t)(lane & 3) * 4u) : "memory");
      if ((w >> lane) & 1u) out[base + __popc(w & lt)] = __uint_as_float(v);
    }
  }
}

// The same accumulator leaving through shared memory: each warp owns a 32-row x 128-byte staging box (128-byte
// swizzle: 16-byte piece j of row r sits at piece j ^ (r & 7), so the 32 row-owning lanes write without bank
// conflicts), fills it from its registers and one lane hands it to the TMA unit, which writes whole lines and clips
// rows >= M and columns >= N.  bf16: 64 columns per box (two tensor-memory reads); fp32: 32 columns per box, the
// K-range index as third coordinate.  Per-thread stores of a row-per-lane layout touch 32 lines per instruction and
// were measured to slow the concurrent main loop by about 15 %.
__device__ __forceinline__ void epilogue_tile_tma(const Params& P, const CUtensorMap* tmC, uint32_t stage, uint32_t tmem_base,
                                                  int acc, int q, int c0, int lane, int64_t m0, int n0, int split) {
  const int64_t row0 = (int64_t)m0 + q * 32;
  const int64_t m = row0 + lane;
  const bool row_ok = m < P.M;
  const uint32_t my_row = stage + (uint32_t)lane * 128u;
  const uint32_t sw = (uint32_t)(lane & 7);
  if (P.epilogue == MST_TC_OUT_BF16) {
#pragma unroll 1
    for (int g = c0; g < BN / 64; g += EPI_WARPS / 4) {
      const int n = n0 + g * 64;
      if (n >= P.N) break;  // uniform
      if (lane == 0) bulk_wait_read();  // the box's previous contents have left shared memory
      __syncwarp();
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int nn = n + h * 32;
        if (nn >= P.N) break;  // uniform; the TMA store clips these columns
        uint32_t r[32];
        uint16_t* pre = reinterpret_cast<uint16_t*>(P.pre) + m * P.ldpre + nn;
        const bool pre_vec = nn + 32 <= P.N && ((P.ldpre & 7) == 0) && ((reinterpret_cast<uintptr_t>(P.pre) & 15u) == 0);
        uint4 p4[4];
        if (P.act == MST_ACT_GELU_GRAD && pre_vec && row_ok) {
#pragma unroll
          for (int v = 0; v < 4; ++v) p4[v] = __ldg(reinterpret_cast<const uint4*>(pre) + v);
        }
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + g * 64 + h * 32), r);
        if (P.act && row_ok) act_chunk(P, r, pre, pre_vec, p4, nn);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const uint32_t piece = (uint32_t)(h * 4 + v) ^ sw;
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(my_row + piece * 16u),
                       "r"(pack_bf16(__uint_as_float(r[8 * v + 0]), __uint_as_float(r[8 * v + 1]))),
                       "r"(pack_bf16(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3]))),
                       "r"(pack_bf16(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5]))),
                       "r"(pack_bf16(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7])))
                       : "memory");
        }
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0 && row0 < P.M) {
        tma_store_2d(tmC, stage, n, (int)row0);
        bulk_commit();
      }
    }
  } else {
#pragma unroll 1
    for (int c = c0; c < BN / 32; c += EPI_WARPS / 4) {
      const int n = n0 + c * 32;
      if (n >= P.N) break;  // uniform
      if (lane == 0) bulk_wait_read();
      __syncwarp();
      uint32_t r[32];
      tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + c * 32), r);
#pragma unroll
      for (int v = 0; v < 8; ++v) {
        const uint32_t piece = (uint32_t)v ^ sw;
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(my_row + piece * 16u), "r"(r[4 * v]), "r"(r[4 * v + 1]),
                     "r"(r[4 * v + 2]), "r"(r[4 * v + 3])
                     : "memory");
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0 && row0 < P.M) {
        tma_store_3d(tmC, stage, n, (int)row0, split);
        bulk_commit();
      }
    }
  }
}

// ------------------------------------------------------------------------------------------- kernel
__global__ void __launch_bounds__(NUM_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmC, const Params P) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
  const uint32_t out_base = tiles_base + STAGES * STAGE_BYTES;  // epilogue staging boxes (1024-byte aligned)
  const uint32_t bar_base = out_base + EPI_WARPS * OUT_BOX_BYTES;
  // barrier slots (8 bytes each): full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]
  const uint32_t full0 = bar_base, empty0 = bar_base + 8 * STAGES, tfull0 = bar_base + 16 * STAGES,
                 tempty0 = tfull0 + 16;
  __shared__ uint32_t tmem_base_holder;
  __shared__ int abort_sh;
  volatile int* abort_flag = &abort_sh;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    abort_sh = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull0 + 8 * a, 1);
      mbar_init(tempty0 + 8 * a, EPI_WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_holder)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_holder;
  mst_grid_launch_dependents();
  mst_grid_dependency_wait();  // set-up above overlaps the predecessor's tail; global memory only from here on

  const int64_t works = (int64_t)P.m_tiles * P.n_tiles * P.splits;
  const int tiles = P.m_tiles * P.n_tiles;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      for (int64_t w = blockIdx.x; w < works && !*abort_flag; w += gridDim.x) {
        const int split = (int)(w / tiles), t = (int)(w % tiles);
        const int m0 = (t / P.n_tiles) * BM, n0 = (t % P.n_tiles) * BN;
        const int kb0 = (int)((int64_t)split * P.kblocks / P.splits), kb1 = (int)((int64_t)(split + 1) * P.kblocks / P.splits);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag)) break;
          const uint32_t fb = full0 + 8 * s;
          const uint32_t sa = tiles_base + s * STAGE_BYTES, sb = sa + A_BYTES;
          mbar_expect_tx(fb, STAGE_BYTES);
          if (P.a_mn) {
            for (int j = 0; j < BM / 64; ++j) tma_load_2d(sa + j * BOX_BYTES, &tmA, m0 + j * 64, kb * BK, fb);
          } else {
            tma_load_2d(sa, &tmA, kb * BK, m0, fb);
          }
          if (P.b_mn) {
            for (int j = 0; j < BN / 64; ++j) tma_load_2d(sb + j * BOX_BYTES, &tmB, n0 + j * 64, kb * BK, fb);
          } else {
            tma_load_2d(sb, &tmB, kb * BK, n0, fb);
          }
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = 256, operand majors
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(P.a_mn ? 1 : 0) << 15) |
                             ((uint32_t)(P.b_mn ? 1 : 0) << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      // The issue loop is one thread's serial instruction stream; everything that does not depend on the stage is
      // formed once here.  K-major: 16 K-elements = 32 bytes further along the swizzled row; MN-major: 16 rows of
      // 128 bytes.
      const uint64_t adesc0 = smem_desc(tiles_base, P.a_mn ? BOX_BYTES : 16, 1024);
      const uint64_t bdesc0 = smem_desc(tiles_base + A_BYTES, P.b_mn ? BOX_BYTES : 16, 1024);
      const uint32_t a_kstep = (uint32_t)(P.a_mn ? UMMA_K * 128 : UMMA_K * 2) >> 4;
      const uint32_t b_kstep = (uint32_t)(P.b_mn ? UMMA_K * 128 : UMMA_K * 2) >> 4;
      int s = 0, acc = 0;
      uint32_t ph = 0, acc_ph = 0;
      for (int64_t w = blockIdx.x; w < works && !*abort_flag; w += gridDim.x) {
        const int split = (int)(w / tiles);
        const int kb0 = (int)((int64_t)split * P.kblocks / P.splits), kb1 = (int)((int64_t)(split + 1) * P.kblocks / P.splits);
        if (!mbar_wait(tempty0 + 8 * acc, acc_ph ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        bool ok = true;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full0 + 8 * s, ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          // descriptors of this stage: the start-address field moves by 16-byte units, nothing else changes
          const uint64_t ad = adesc0 + (uint64_t)(uint32_t)(s * (STAGE_BYTES >> 4));
          const uint64_t bd = bdesc0 + (uint64_t)(uint32_t)(s * (STAGE_BYTES >> 4));
          tc_mma(d_tmem, ad, bd, idesc, kb > kb0 ? 1u : 0u);
#pragma unroll
          for (int k = 1; k < BK / UMMA_K; ++k) tc_mma(d_tmem, ad + (uint64_t)(k * a_kstep), bd + (uint64_t)(k * b_kstep), idesc, 1u);
          tc_commit(empty0 + 8 * s);  // the smem stage is free once these MMAs have read it
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull0 + 8 * acc);  // accumulator complete
        if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    const int q = warp & 3;  // tensor-memory lane quarter this warp may read
    const bool use_tma = P.tma_out && P.epilogue != MST_TC_OUT_SAMPLED;
    int acc = 0;
    uint32_t acc_ph = 0;
    for (int64_t w = blockIdx.x; w < works; w += gridDim.x) {
      const int split = (int)(w / tiles), t = (int)(w % tiles);
      const int m0 = (t / P.n_tiles) * BM, n0 = (t % P.n_tiles) * BN;
      if (!mbar_wait(tfull0 + 8 * acc, acc_ph, abort_flag)) break;
      tc_fence_after();
      if (use_tma)
        epilogue_tile_tma(P, &tmC, out_base + (uint32_t)(warp - 2) * OUT_BOX_BYTES, tmem_base, acc, q, (warp - 2) >> 2, lane, m0,
                          n0, split);
      else if (P.epilogue == MST_TC_OUT_SAMPLED)
        epilogue_tile_sampled(P, out_base + (uint32_t)(warp - 2) * OUT_BOX_BYTES, tmem_base, acc, q, (warp - 2) >> 2, lane, m0,
                              n0, split);
      else
        epilogue_tile(P, tmem_base, acc, q, (warp - 2) >> 2, lane, m0, n0, split);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
      if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
    }
    if (use_tma && lane == 0) bulk_wait_all();  // this warp's stores have landed before shared memory is given back
  }

  // ------------------------------------------------------------------ teardown
  if (*abort_flag) {
    // give copies and MMAs already in flight time to land before shared and tensor memory are released
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------------------------------- CTA-pair kernel
// Same roles, but two blocks of a cluster (an SM pair) share one 256 x 256 output tile: each block loads its own 128
// rows of A and its own half (128 of 256 columns) of B, the even block issues tcgen05.mma.cta_group::2 (M = 256) that
// reads both blocks' shared memory and writes both blocks' tensor memory.  Per block this halves the shared-memory
// traffic for B, which is what bounds the single-block kernel.  Barrier protocol:
//   full[s]   (even block)  two arrivals (one per block's producer, each announcing its own bytes) + TMA bytes of both
//   empty[s]  (each block)  one arrival, multicast by the even block's tcgen05.commit
//   tfull[a]  (each block)  one arrival, multicast by tcgen05.commit after the tile's last MMA
//   tempty[a] (even block)  sixteen arrivals: the eight epilogue warps of both blocks
constexpr int P_STAGES = 6;
constexpr int PB_BYTES = (BN / 2) * BK * 2;        // this block's half of B: 16 KiB
constexpr int P_STAGE_BYTES = A_BYTES + PB_BYTES;  // 32 KiB
constexpr size_t P_SMEM_BYTES = (size_t)P_STAGES * P_STAGE_BYTES + EPI_WARPS * OUT_BOX_BYTES + 1024 + 256;
// shared::cluster address of the same shared-memory location in the even block (rank 0) of the pair
__device__ __forceinline__ uint32_t in_even_block(uint32_t local_addr) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(0u));
  return r;
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(tm), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"((uint16_t)3)
               : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
tc_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmC, const Params P) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;
  const uint32_t out_base = tiles_base + P_STAGES * P_STAGE_BYTES;
  const uint32_t bar_base = out_base + EPI_WARPS * OUT_BOX_BYTES;
  const uint32_t full0 = bar_base, empty0 = bar_base + 8 * P_STAGES, tfull0 = bar_base + 16 * P_STAGES,
                 tempty0 = tfull0 + 16;
  __shared__ uint32_t tmem_base_holder;
  __shared__ int abort_sh;
  volatile int* abort_flag = &abort_sh;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = even block (issues the MMAs), 1 = its peer
  if (threadIdx.x == 0) {
    abort_sh = 0;
    for (int s = 0; s < P_STAGES; ++s) {
      mbar_init(full0 + 8 * s, 2);
      mbar_init(empty0 + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull0 + 8 * a, 1);
      mbar_init(tempty0 + 8 * a, 2 * EPI_WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_holder)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both blocks' barriers are initialised before any remote arrival or copy completion
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_holder;
  mst_grid_launch_dependents();
  mst_grid_dependency_wait();

  const int m_pairs = (P.m_tiles + 1) / 2;
  const int tiles = m_pairs * P.n_tiles;
  const int64_t works = (int64_t)tiles * P.splits;
  const int64_t pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer (both blocks)
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      for (int64_t w = pair; w < works && !*abort_flag; w += npairs) {
        const int split = (int)(w / tiles), t = (int)(w % tiles);
        const int m0 = (t / P.n_tiles) * (2 * BM) + (int)rank * BM;       // this block's rows
        const int n0 = (t % P.n_tiles) * BN + (int)rank * (BN / 2);       // this block's half of B
        const int kb0 = (int)((int64_t)split * P.kblocks / P.splits), kb1 = (int)((int64_t)(split + 1) * P.kblocks / P.splits);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag)) break;
          const uint32_t fb = in_even_block(full0 + 8 * s);  // the even block's barrier collects both blocks' bytes
          const uint32_t sa = tiles_base + s * P_STAGE_BYTES, sb = sa + A_BYTES;
          mbar_expect_tx_cluster(fb, P_STAGE_BYTES);
          if (P.a_mn) {
            for (int j = 0; j < BM / 64; ++j) tma_load_2d_pair(sa + j * BOX_BYTES, &tmA, m0 + j * 64, kb * BK, fb);
          } else {
            tma_load_2d_pair(sa, &tmA, kb * BK, m0, fb);
          }
          if (P.b_mn) {
            for (int j = 0; j < BN / 128; ++j) tma_load_2d_pair(sb + j * BOX_BYTES, &tmB, n0 + j * 64, kb * BK, fb);
          } else {
            tma_load_2d_pair(sb, &tmB, kb * BK, n0, fb);
          }
          if (++s == P_STAGES) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (even block only)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(P.a_mn ? 1 : 0) << 15) |
                             ((uint32_t)(P.b_mn ? 1 : 0) << 16) | ((uint32_t)(BN >> 3) << 17) |
                             ((uint32_t)((2 * BM) >> 4) << 24);
      const uint64_t adesc0 = smem_desc(tiles_base, P.a_mn ? BOX_BYTES : 16, 1024);
      const uint64_t bdesc0 = smem_desc(tiles_base + A_BYTES, P.b_mn ? BOX_BYTES : 16, 1024);
      const uint32_t a_kstep = (uint32_t)(P.a_mn ? UMMA_K * 128 : UMMA_K * 2) >> 4;
      const uint32_t b_kstep = (uint32_t)(P.b_mn ? UMMA_K * 128 : UMMA_K * 2) >> 4;
      int s = 0, acc = 0;
      uint32_t ph = 0, acc_ph = 0;
      for (int64_t w = pair; w < works && !*abort_flag; w += npairs) {
        const int split = (int)(w / tiles);
        const int kb0 = (int)((int64_t)split * P.kblocks / P.splits), kb1 = (int)((int64_t)(split + 1) * P.kblocks / P.splits);
        if (!mbar_wait(tempty0 + 8 * acc, acc_ph ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        bool ok = true;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full0 + 8 * s, ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          // descriptors of this stage: the start-address field moves by 16-byte units, nothing else changes
          const uint64_t ad = adesc0 + (uint64_t)(uint32_t)(s * (P_STAGE_BYTES >> 4));
          const uint64_t bd = bdesc0 + (uint64_t)(uint32_t)(s * (P_STAGE_BYTES >> 4));
          tc_mma_pair(d_tmem, ad, bd, idesc, kb > kb0 ? 1u : 0u);
#pragma unroll
          for (int k = 1; k < BK / UMMA_K; ++k) tc_mma_pair(d_tmem, ad + (uint64_t)(k * a_kstep), bd + (uint64_t)(k * b_kstep), idesc, 1u);
          tc_commit_pair(empty0 + 8 * s);  // frees this stage in both blocks
          if (++s == P_STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair(tfull0 + 8 * acc);  // both blocks' halves of the accumulator are complete
        if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (both blocks, own 128 rows)
    const int q = warp & 3;
    const bool use_tma = P.tma_out && P.epilogue != MST_TC_OUT_SAMPLED;
    int acc = 0;
    uint32_t acc_ph = 0;
    for (int64_t w = pair; w < works; w += npairs) {
      const int split = (int)(w / tiles), t = (int)(w % tiles);
      const int m0 = (t / P.n_tiles) * (2 * BM) + (int)rank * BM, n0 = (t % P.n_tiles) * BN;
      if (!mbar_wait(tfull0 + 8 * acc, acc_ph, abort_flag)) break;
      tc_fence_after();
      if (use_tma)
        epilogue_tile_tma(P, &tmC, out_base + (uint32_t)(warp - 2) * OUT_BOX_BYTES, tmem_base, acc, q, (warp - 2) >> 2, lane, m0,
                          n0, split);
      else if (P.epilogue == MST_TC_OUT_SAMPLED)
        epilogue_tile_sampled(P, out_base + (uint32_t)(warp - 2) * OUT_BOX_BYTES, tmem_base, acc, q, (warp - 2) >> 2, lane, m0,
                              n0, split);
      else
        epilogue_tile(P, tmem_base, acc, q, (warp - 2) >> 2, lane, m0, n0, split);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(in_even_block(tempty0 + 8 * acc));
      if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
    }
    if (use_tma && lane == 0) bulk_wait_all();  // this warp's stores have landed before shared memory is given back
  }

  // ------------------------------------------------------------------ teardown
  if (*abort_flag) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer may still be signalling this block's barriers or reading its shared memory
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// out[i] = sum over splits of partial[s][i], fixed order
__global__ void tc_reduce_kernel(const float* __restrict__ partial, int splits, int64_t n, float* __restrict__ out) {
  mst_grid_launch_dependents();
  mst_grid_dependency_wait();
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float s = partial[i];
  for (int k = 1; k < splits; ++k) s += partial[(int64_t)k * n + i];
  out[i] = s;
}

// the same, four values per thread (n a multiple of 4, 16-byte aligned pointers)
__global__ void tc_reduce4_kernel(const float4* __restrict__ partial, int splits, int64_t n4, float4* __restrict__ out) {
  mst_grid_launch_dependents();
  mst_grid_dependency_wait();
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  float4 s = partial[i];
  for (int k = 1; k < splits; ++k) {
    const float4 v = partial[(int64_t)k * n4 + i];
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
  }
  out[i] = s;
}

// ------------------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// rows x cols (cols contiguous, ld elements between rows) bf16 matrix; box = box_rows x 64 columns
bool make_map(CUtensorMap* tm, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1u, 1u};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Output maps for the staged epilogue.  bf16 [M x N] (ld elements between rows), box 64 columns x 32 rows;
// fp32 [splits x M x N], box 32 columns x 32 rows x 1.  Both boxes are 128 bytes wide (128-byte swizzle).
bool make_out_map_bf16(CUtensorMap* tm, void* base, int64_t M, int64_t N, int64_t ld) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || (ld % 8) != 0 || (reinterpret_cast<uintptr_t>(base) & 15u) != 0) return false;
  cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64u, 32u};
  cuuint32_t estr[2] = {1u, 1u};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
bool make_out_map_f32(CUtensorMap* tm, void* base, int64_t M, int64_t N, int64_t ld, int64_t slab_elems, int splits) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || (ld % 4) != 0 || (slab_elems % 4) != 0 || (reinterpret_cast<uintptr_t>(base) & 15u) != 0) return false;
  cuuint64_t dims[3] = {(cuuint64_t)N, (cuuint64_t)M, (cuuint64_t)splits};
  cuuint64_t strides[2] = {(cuuint64_t)ld * 4, (cuuint64_t)slab_elems * 4};
  cuuint32_t box[3] = {32u, 32u, 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
  static int n[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return 148;
  if (!n[dev]) {
    if (cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n[dev] <= 0) n[dev] = 148;
  }
  return n[dev];
}

}  // namespace

// Number of K ranges for a contraction whose output has few tiles: minimise a simple time model
//   waves * (k-blocks per range * t_kblock + t_tile) + traffic of the partial sums
// over 1..16 ranges.  `works1` = tile jobs with one range, `slots` = jobs that run at once (blocks or block pairs),
// `out_bytes` = bytes one range writes as partial sums (and the reduction reads back).
int mst_tc_pick_splits(int64_t works1, int64_t slots, int64_t kblocks, double out_bytes) {
  const double t_kblock = 0.32e-6, t_tile = 1.5e-6, bw = 4.0e12, t_reduce_launch = 3.0e-6;
  int best = 1;
  double best_t = 1e30;
  for (int sp = 1; sp <= 16 && sp <= kblocks; ++sp) {
    const int64_t waves = (works1 * sp + slots - 1) / slots;
    const double kb = (double)((kblocks + sp - 1) / sp);
    double t = (double)waves * (kb * t_kblock + t_tile);
    if (sp > 1) t += t_reduce_launch + (double)sp * out_bytes * 2.0 / bw;
    if (t < best_t * 0.97) {  // prefer fewer ranges unless the gain is clear
      best_t = t;
      best = sp;
    }
  }
  return best;
}

// Per-device scratch buffers, grown on demand (growing waits for the device and frees the old buffer).
//   MST_WS_SPLIT    partial sums of a K-range split.  Every call that splits its contraction range shares its device's
//                   buffer, so two such calls must not overlap on the GPU (mst_dense_grad, mst_dense_grad_dw,
//                   mst_sddmm_dw and the host-step calls on the tensor path): keep them on one stream or order them
//                   with events.
//   MST_WS_COLUMNS  feature-major copies of activations for the structured-sparse path and the CUDA-core kernels
//                   (same rule).
//   MST_WS_ATTENTION  per-row dot products of the attention backward pass (same rule).
//   MST_WS_IMAGE    dense bf16 image of W.M of the layer being multiplied, for layers without value tracking
//                   (same rule).
mst_status_t mst_workspace_kind(int kind, size_t bytes, void** ptr) {
  constexpr int MAX_DEVICES = 64;
  static void* buf[MST_WS_KINDS][MAX_DEVICES] = {};
  static size_t cap[MST_WS_KINDS][MAX_DEVICES] = {};
  int dev = 0;
  MST_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEVICES || kind < 0 || kind >= MST_WS_KINDS) return MST_ERR_CUDA;
  if (bytes > cap[kind][dev]) {
    if (buf[kind][dev]) {
      MST_CUDA_TRY(cudaDeviceSynchronize());
      MST_CUDA_TRY(cudaFree(buf[kind][dev]));
      buf[kind][dev] = nullptr;
      cap[kind][dev] = 0;
    }
    const size_t want = (bytes + ((size_t)1 << 20)) & ~(((size_t)1 << 20) - 1);
    MST_CUDA_TRY(cudaMalloc(&buf[kind][dev], want));
    cap[kind][dev] = want;
  }
  *ptr = buf[kind][dev];
  return MST_OK;
}
mst_status_t mst_workspace(size_t bytes, void** ptr) { return mst_workspace_kind(MST_WS_SPLIT, bytes, ptr); }

bool mst_tc_gemm_usable(const void* A, int64_t lda, const void* B, int64_t ldb) {
  return (lda % 8 == 0) && (ldb % 8 == 0) && ((reinterpret_cast<uintptr_t>(A) & 15u) == 0) &&
         ((reinterpret_cast<uintptr_t>(B) & 15u) == 0) && encode_fn() != nullptr;
}

mst_status_t mst_tc_gemm(const mst_tc_gemm_args& a, cudaStream_t s) {
  if (a.M <= 0 || a.N <= 0 || a.K <= 0) return MST_ERR_INVALID_ARG;
  if (!mst_tc_gemm_usable(a.A, a.lda, a.B, a.ldb)) return MST_ERR_SHAPE;
  CUtensorMap tmA, tmB;
  // Block pairs (256-row tiles) pay off once there are at least two row tiles; MST_TC_PAIR=0/1 overrides.
  bool pair = a.M > BM;
  if (const char* e = getenv("MST_TC_PAIR")) pair = (e[0] == '1');
  // K-major: [rows x K], box 64 (K) x tile rows.  MN-major: [K x rows], box 64 (rows) x BK.
  const bool okA = a.a_mn_major ? make_map(&tmA, a.A, a.K, a.M, a.lda, BK) : make_map(&tmA, a.A, a.M, a.K, a.lda, BM);
  const int b_rows = pair ? BN / 2 : BN;
  const bool okB = a.b_mn_major ? make_map(&tmB, a.B, a.K, a.N, a.ldb, BK) : make_map(&tmB, a.B, a.N, a.K, a.ldb, b_rows);
  if (!okA || !okB) return MST_ERR_SHAPE;
  Params P;
  P.M = a.M;
  P.N = a.N;
  P.kblocks = (int)((a.K + BK - 1) / BK);
  P.splits = 1;
  P.m_tiles = (int)((a.M + BM - 1) / BM);
  P.n_tiles = (int)((a.N + BN - 1) / BN);
  P.a_mn = a.a_mn_major;
  P.b_mn = a.b_mn_major;
  P.epilogue = a.epilogue;
  P.out = a.out;
  P.ldc = a.ldc;
  P.partial = nullptr;
  P.bits = a.bits;
  P.wscan = a.wscan;
  P.wpr = a.wpr;
  P.nnz = a.nnz;
  P.act = a.epilogue == MST_TC_OUT_BF16 ? a.act : 0;
  P.pre = a.pre;
  P.ldpre = a.ldpre;
  if (P.act == MST_ACT_GELU_GRAD && !P.pre) return MST_ERR_INVALID_ARG;
  P.sampled_stage_min = 384;  // measured: row-by-row stores pay from a density of about 0.4
  if (const char* e = getenv("MST_TC_SAMPLED_STAGE")) P.sampled_stage_min = atoi(e);  // measurement override
  if (a.epilogue != MST_TC_OUT_BF16) {
    // few output tiles: cut the contraction range so that all SMs work; partial sums go to the shared scratch buffer
    const int64_t works1 = pair ? (int64_t)((P.m_tiles + 1) / 2) * P.n_tiles : (int64_t)P.m_tiles * P.n_tiles;
    const int64_t slots = pair ? sm_count() / 2 : sm_count();
    const double out_bytes = a.epilogue == MST_TC_OUT_F32 ? 4.0 * (double)a.M * (double)a.N : 4.0 * (double)a.nnz;
    P.splits = a.splits > 0 ? a.splits : mst_tc_pick_splits(works1, slots, P.kblocks, out_bytes);
    if (const char* e = getenv("MST_TC_SPLITS")) {  // measurement override
      const int v = atoi(e);
      if (v > 0) P.splits = v;
    }
    if (P.splits > P.kblocks) P.splits = P.kblocks;
    if (P.splits > 1) {
      const size_t per = a.epilogue == MST_TC_OUT_F32 ? (size_t)a.M * a.N : (size_t)a.nnz;
      void* ws = nullptr;
      MST_TRY(mst_workspace(sizeof(float) * per * P.splits, &ws));
      P.partial = (float*)ws;
    }
  }
  // staged epilogue when the output can be described to the TMA unit (MST_TC_TMA_OUT=0 keeps per-thread stores)
  CUtensorMap tmC = tmA;
  P.tma_out = 0;
  if (a.epilogue == MST_TC_OUT_BF16) {
    P.tma_out = make_out_map_bf16(&tmC, a.out, a.M, a.N, a.ldc) ? 1 : 0;
  } else if (a.epilogue == MST_TC_OUT_F32) {
    P.tma_out = (P.splits > 1 ? make_out_map_f32(&tmC, P.partial, a.M, a.N, a.N, a.M * a.N, P.splits)
                              : make_out_map_f32(&tmC, a.out, a.M, a.N, a.ldc, a.M * a.ldc, 1))
                    ? 1
                    : 0;
  }
  if (const char* e = getenv("MST_TC_TMA_OUT")) {
    if (e[0] == '0') P.tma_out = 0;
  }
  if (pair) {
    MST_CUDA_TRY(cudaFuncSetAttribute(tc_gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)P_SMEM_BYTES));
    const int64_t works = (int64_t)((P.m_tiles + 1) / 2) * P.n_tiles * P.splits;
    const int64_t max_pairs = sm_count() / 2;
    const int grid = 2 * (int)(works < max_pairs ? works : max_pairs);
    MST_CUDA_TRY(mst_launch_overlapped(tc_gemm_pair_kernel, dim3(grid), dim3(NUM_THREADS), P_SMEM_BYTES, s, tmA, tmB, tmC, P));
  } else {
    MST_CUDA_TRY(cudaFuncSetAttribute(tc_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    const int64_t works = (int64_t)P.m_tiles * P.n_tiles * P.splits;
    const int grid = (int)(works < sm_count() ? works : sm_count());
    MST_CUDA_TRY(mst_launch_overlapped(tc_gemm_kernel, dim3(grid), dim3(NUM_THREADS), SMEM_BYTES, s, tmA, tmB, tmC, P));
  }
  MST_CUDA_TRY(cudaGetLastError());
  if (P.splits > 1) {
    const int64_t n = a.epilogue == MST_TC_OUT_F32 ? a.M * a.N : a.nnz;
    if (n > 0 && (n & 3) == 0 && (reinterpret_cast<uintptr_t>(a.out) & 15u) == 0)
      MST_CUDA_TRY(mst_launch_overlapped(tc_reduce4_kernel, dim3((unsigned)((n / 4 + 255) / 256)), dim3(256), 0, s,
                                         (const float4*)P.partial, P.splits, n / 4, (float4*)a.out));
    else if (n > 0)
      MST_CUDA_TRY(mst_launch_overlapped(tc_reduce_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, s,
                                         (const float*)P.partial, P.splits, n, (float*)a.out));
    MST_CUDA_TRY(cudaGetLastError());
  }
  return MST_OK;
}

extern "C" mst_status_t mst_device_error_flags(int32_t* flags) {
  if (!flags) return MST_ERR_INVALID_ARG;
  int v = 0;
  MST_CUDA_TRY(cudaDeviceSynchronize());
  MST_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_tc_error, sizeof(int)));
  int32_t att = 0;
  MST_TRY(mst_attention_error_flags(&att));
  int32_t sp = 0, cc = 0;
  MST_TRY(mst_sp24_error_flags(&sp));
  MST_TRY(mst_spmm_error_flags(&cc));
  int32_t sd = 0;
  MST_TRY(mst_sddmm_error_flags(&sd));
  cc |= sd;
  *flags = v | (att << 1) | (sp << 2) | (cc << 3);
  return MST_OK;
}
