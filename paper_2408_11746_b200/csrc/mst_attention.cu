// Strided sparse self-attention, forward (Sec. 3.3: position i attends to j <= i with i - j < l, and to every l-th
// earlier position j = i - l, i - 2l, ...; every head uses the same pattern).
//
// One block per (batch, head, 128 queries).  The window part is two dense tensor-core products on a [128 x (l+128)]
// score tile: the keys q0 - l .. q0 + 127 cover the window of every query of the block, so no loop over key blocks
// and no running softmax is needed:
//   control warp   TMA loads Q, the l/128 + 1 key blocks and value blocks; tcgen05.mma S = Q K^T (fp32, tensor
//                  memory); after the softmax warps have written P, tcgen05.mma O = P V;
//   4 softmax warps (thread = query row = tensor-memory lane): scores of the strided positions on CUDA cores
//                  (at most n/l - 1 dot products of 64), row maximum and sum over tensor memory, P in bf16 into
//                  shared memory in the K-major 128-byte-swizzled operand layout, then O / sum plus the strided
//                  positions' values, written as bf16.
// Keys before the start of the sequence (q0 < l) are fetched from the rows in front of it (another sequence of the
// batch, or the TMA unit's zero fill before row 0) and masked by position, never by value.
// Every mbarrier wait is bounded (abort flag + sticky error word), as in the contraction kernel.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "mst_internal.cuh"
#include "mst_tc_ptx.cuh"

namespace {

using namespace mst_ptx;

constexpr int D = 64;          // head dimension
constexpr int BQ = 128;        // queries per block = tensor-memory lanes
constexpr int KB = 128;        // keys per key block
constexpr int TILE_BYTES = 128 * D * 2;  // one [128 x 64] bf16 tile, 16 KiB
constexpr int ATT_THREADS = 160;         // 4 softmax warps + 1 control warp
constexpr int TMEM_COLS = 512;
constexpr int O_COL = 448;     // output accumulator: tensor-memory columns 448..511
constexpr int MAX_EXTRA = 15;  // strided positions per query: seq / l - 1

__device__ int g_attn_error = 0;

struct AttnParams {
  const uint16_t *Q, *K, *V;
  int64_t ld;       // elements between consecutive tokens in Q / K / V
  uint16_t* out;
  int64_t ldo;
  float* lse;       // [batch, heads, seq] or NULL
  int seq, heads, stride;
  int nkb;          // key blocks per tile: stride / 128 + 1
};

__device__ __forceinline__ bool att_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return mst_ptx::mbar_wait(bar, parity, abort_flag, &g_attn_error);
}

__device__ __forceinline__ float ex2_ftz(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ float dot8(const uint4& a, const uint4& b, float acc) {
  acc = fmaf(bf_lo(a.x), bf_lo(b.x), acc); acc = fmaf(bf_hi(a.x), bf_hi(b.x), acc);
  acc = fmaf(bf_lo(a.y), bf_lo(b.y), acc); acc = fmaf(bf_hi(a.y), bf_hi(b.y), acc);
  acc = fmaf(bf_lo(a.z), bf_lo(b.z), acc); acc = fmaf(bf_hi(a.z), bf_hi(b.z), acc);
  acc = fmaf(bf_lo(a.w), bf_lo(b.w), acc); acc = fmaf(bf_hi(a.w), bf_hi(b.w), acc);
  return acc;
}

__global__ void __launch_bounds__(ATT_THREADS, 1)
strided_attention_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                             const __grid_constant__ CUtensorMap tmV, const AttnParams P) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int nkb = P.nkb;
  const uint32_t q_s = base, k_s = q_s + TILE_BYTES, v_s = k_s + nkb * TILE_BYTES, p_s = v_s + nkb * TILE_BYTES;
  const uint32_t bar0 = p_s + 2 * nkb * TILE_BYTES;
  const uint32_t bar_qk = bar0, bar_v = bar0 + 8, bar_s = bar0 + 16, bar_p = bar0 + 24, bar_o = bar0 + 32;
  __shared__ uint32_t tmem_base_holder;
  __shared__ int abort_sh;
  volatile int* abort_flag = &abort_sh;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = blockIdx.x * BQ, h = blockIdx.y, b = blockIdx.z;
  const int l = P.stride;
  const int jb = q0 - l;                               // first key of the tile (may be negative)
  const int64_t row_base = (int64_t)b * P.seq;         // first token of this sequence

  if (threadIdx.x == 0) {
    abort_sh = 0;
    mbar_init(bar_qk, 1);
    mbar_init(bar_v, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_p, 4);
    mbar_init(bar_o, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_holder)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_holder;

  if (warp == 4) {
    // ------------------------------------------------------------------ control: loads and the two products
    if (lane == 0) {
      const int col = h * D;
      mbar_expect_tx(bar_qk, (uint32_t)((1 + nkb) * TILE_BYTES));
      tma_load_2d(q_s, &tmQ, col, (int)(row_base + q0), bar_qk);
      for (int kb = 0; kb < nkb; ++kb) tma_load_2d(k_s + kb * TILE_BYTES, &tmK, col, (int)(row_base + jb + kb * KB), bar_qk);
      mbar_expect_tx(bar_v, (uint32_t)(nkb * TILE_BYTES));
      for (int kb = 0; kb < nkb; ++kb) tma_load_2d(v_s + kb * TILE_BYTES, &tmV, col, (int)(row_base + jb + kb * KB), bar_v);

      bool ok = att_wait(bar_qk, 0, abort_flag);
      if (ok) {
        tc_fence_after();
        // S[:, kb*128 .. +128) = Q K_kb^T : M = 128, N = 128, both operands K-major, four K steps of 16
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(KB >> 3) << 17) | ((uint32_t)(BQ >> 4) << 24);
        const uint64_t qd = smem_desc(q_s, 16, 1024);
        for (int kb = 0; kb < nkb; ++kb) {
          const uint64_t kd = smem_desc(k_s + kb * TILE_BYTES, 16, 1024);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            tc_mma(tmem_base + (uint32_t)(kb * KB), qd + (uint64_t)(ks * 2), kd + (uint64_t)(ks * 2), idesc, ks > 0 ? 1u : 0u);
        }
        tc_commit(bar_s);
        ok = att_wait(bar_v, 0, abort_flag) && att_wait(bar_p, 0, abort_flag);
      }
      if (ok) {
        tc_fence_after();
        // O = P V : M = 128, N = 64, P K-major (64-key blocks of 16 KiB), V as stored (keys x 64: MN-major)
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(D >> 3) << 17) |
                               ((uint32_t)(BQ >> 4) << 24);
        const int ksteps = nkb * KB / 16;
        for (int ks = 0; ks < ksteps; ++ks) {
          const uint64_t pd = smem_desc(p_s + (uint32_t)(ks >> 2) * TILE_BYTES + (uint32_t)(ks & 3) * 32u, 16, 1024);
          const uint64_t vd = smem_desc(v_s + (uint32_t)ks * (16u * 128u), 8192, 1024);
          tc_mma(tmem_base + (uint32_t)O_COL, pd, vd, idesc, ks > 0 ? 1u : 0u);
        }
        tc_commit(bar_o);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax: thread = query row
    const int r = warp * 32 + lane;
    const int i = q0 + r;                               // position in the sequence
    const int64_t tok = row_base + i;
    const float c = 0.125f * 1.4426950408889634f;       // log2(e) / sqrt(64)
    const int n_ext = i / l < MAX_EXTRA ? i / l : MAX_EXTRA;
    const uint4* qrow = reinterpret_cast<const uint4*>(P.Q + tok * P.ld + h * D);
    float s_ext[MAX_EXTRA];
#pragma unroll 1
    for (int k = 0; k < n_ext; ++k) {
      const uint4* krow = reinterpret_cast<const uint4*>(P.K + (tok - (int64_t)(k + 1) * l) * P.ld + h * D);
      float acc = 0.f;
#pragma unroll
      for (int v = 0; v < 8; ++v) acc = dot8(__ldg(qrow + v), __ldg(krow + v), acc);
      s_ext[k] = acc;
    }
    float m = -INFINITY;
#pragma unroll 1
    for (int k = 0; k < n_ext; ++k) m = fmaxf(m, s_ext[k]);

    // chunks of 32 keys that hold a visible key for some row of this warp
    const int i_lo = q0 + warp * 32, i_hi = i_lo + 31;
    const int nchunks = nkb * 4;
    bool ok = att_wait(bar_s, 0, abort_flag);
    tc_fence_after();
    if (ok) {
      // pass 1: row maximum
#pragma unroll 1
      for (int ch = 0; ch < nchunks; ++ch) {
        const int j0 = jb + ch * 32;
        if (j0 > i_hi || j0 + 31 <= i_lo - l || j0 + 31 < 0) continue;  // uniform over the warp: nothing visible
        uint32_t v[32];
        tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(ch * 32), v);
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const int j = j0 + e;
          const bool vis = j >= 0 && j <= i && i - j < l;
          m = fmaxf(m, vis ? __uint_as_float(v[e]) : -INFINITY);
        }
      }
      // pass 2: P = exp(s - m) in bf16 into the operand layout, row sum in fp32
      float sum = 0.f;
      const float mc = m * c;
#pragma unroll 1
      for (int ch = 0; ch < nchunks; ++ch) {
        const int j0 = jb + ch * 32;
        const uint32_t prow = p_s + (uint32_t)(ch >> 1) * TILE_BYTES + (uint32_t)r * 128u;
        const uint32_t piece0 = (uint32_t)(ch & 1) * 4u;
        const uint32_t sw = (uint32_t)(r & 7);
        if (j0 > i_hi || j0 + 31 <= i_lo - l || j0 + 31 < 0) {
#pragma unroll
          for (int q = 0; q < 4; ++q)
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(prow + (((piece0 + q) ^ sw) << 4)), "r"(0u) : "memory");
          continue;
        }
        uint32_t v[32];
        tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(ch * 32), v);
        float p[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const int j = j0 + e;
          const bool vis = j >= 0 && j <= i && i - j < l;
          p[e] = vis ? ex2_ftz(fmaf(__uint_as_float(v[e]), c, -mc)) : 0.f;
          sum += p[e];
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(prow + (((piece0 + q) ^ sw) << 4)),
                       "r"(pack_bf16(p[8 * q + 0], p[8 * q + 1])), "r"(pack_bf16(p[8 * q + 2], p[8 * q + 3])),
                       "r"(pack_bf16(p[8 * q + 4], p[8 * q + 5])), "r"(pack_bf16(p[8 * q + 6], p[8 * q + 7]))
                       : "memory");
      }
      // strided positions' weights (kept in fp32, applied on CUDA cores below)
#pragma unroll 1
      for (int k = 0; k < n_ext; ++k) {
        s_ext[k] = ex2_ftz(fmaf(s_ext[k], c, -mc));
        sum += s_ext[k];
      }
      fence_async_smem();  // P is read by the tensor core through the async proxy
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p);

      if (P.lse) P.lse[((int64_t)b * P.heads + h) * P.seq + i] = m * 0.125f + __logf(sum);

      ok = att_wait(bar_o, 0, abort_flag);
      tc_fence_after();
      if (ok) {
        const float inv = 1.0f / sum;
        uint16_t* orow = P.out + tok * P.ldo + h * D;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          uint32_t v[32];
          tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(O_COL + half * 32), v);
          float o[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = __uint_as_float(v[e]);
#pragma unroll 1
          for (int k = 0; k < n_ext; ++k) {
            const uint4* vrow = reinterpret_cast<const uint4*>(P.V + (tok - (int64_t)(k + 1) * l) * P.ld + h * D) + half * 4;
            const float pk = s_ext[k];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint4 x = __ldg(vrow + q);
              o[8 * q + 0] = fmaf(pk, bf_lo(x.x), o[8 * q + 0]); o[8 * q + 1] = fmaf(pk, bf_hi(x.x), o[8 * q + 1]);
              o[8 * q + 2] = fmaf(pk, bf_lo(x.y), o[8 * q + 2]); o[8 * q + 3] = fmaf(pk, bf_hi(x.y), o[8 * q + 3]);
              o[8 * q + 4] = fmaf(pk, bf_lo(x.z), o[8 * q + 4]); o[8 * q + 5] = fmaf(pk, bf_hi(x.z), o[8 * q + 5]);
              o[8 * q + 6] = fmaf(pk, bf_lo(x.w), o[8 * q + 6]); o[8 * q + 7] = fmaf(pk, bf_hi(x.w), o[8 * q + 7]);
            }
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint4 w;
            w.x = pack_bf16(o[8 * q + 0] * inv, o[8 * q + 1] * inv);
            w.y = pack_bf16(o[8 * q + 2] * inv, o[8 * q + 3] * inv);
            w.z = pack_bf16(o[8 * q + 4] * inv, o[8 * q + 5] * inv);
            w.w = pack_bf16(o[8 * q + 6] * inv, o[8 * q + 7] * inv);
            reinterpret_cast<uint4*>(orow)[half * 4 + q] = w;
          }
        }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  if (*abort_flag) {
    for (int t = 0; t < 2000; ++t) __nanosleep(1000);  // let copies and MMAs in flight land
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn att_encode_fn() {
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

// [rows x cols] bf16, ld elements between rows; box = 128 rows x 64 columns (one head of one block of tokens)
bool att_map(CUtensorMap* tm, const void* base, int64_t rows, int64_t cols, int64_t ld) {
  EncodeTiledFn fn = att_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)D, 128u};
  cuuint32_t estr[2] = {1u, 1u};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

mst_status_t mst_attention_error_flags(int32_t* flags) {
  int v = 0;
  MST_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_attn_error, sizeof(int)));
  *flags = v;
  return MST_OK;
}

extern "C" mst_status_t mst_strided_attention_fwd(const void* Q, const void* K, const void* V, int64_t ld, int32_t batch,
                                                  int32_t seq_len, int32_t heads, int32_t head_dim, int32_t stride,
                                                  void* Out, int64_t ldo, float* lse, mst_stream_t stream) {
  if (!Q || !K || !V || !Out || batch < 0 || seq_len <= 0 || heads <= 0) return MST_ERR_INVALID_ARG;
  if (head_dim != D || seq_len % BQ != 0 || stride <= 0 || stride % KB != 0 || stride + KB > O_COL) return MST_ERR_SHAPE;
  if (seq_len / stride - 1 > MAX_EXTRA) return MST_ERR_SHAPE;
  const int64_t width = (int64_t)heads * D;
  if (ld < width || ldo < width || ld % 8 != 0 || ldo % 8 != 0) return MST_ERR_SHAPE;
  if (((reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V) |
        reinterpret_cast<uintptr_t>(Out)) & 15u) != 0)
    return MST_ERR_SHAPE;
  if (batch == 0) return MST_OK;
  const int64_t rows = (int64_t)batch * seq_len;
  if (rows > 0x7FFFFFFF) return MST_ERR_SHAPE;
  CUtensorMap tmQ, tmK, tmV;
  if (!att_map(&tmQ, Q, rows, width, ld) || !att_map(&tmK, K, rows, width, ld) || !att_map(&tmV, V, rows, width, ld))
    return MST_ERR_SHAPE;
  AttnParams P;
  P.Q = (const uint16_t*)Q; P.K = (const uint16_t*)K; P.V = (const uint16_t*)V;
  P.ld = ld;
  P.out = (uint16_t*)Out;
  P.ldo = ldo;
  P.lse = lse;
  P.seq = seq_len; P.heads = heads; P.stride = stride;
  P.nkb = stride / KB + 1;
  const size_t smem = (size_t)(1 + 4 * P.nkb) * TILE_BYTES + 1024 + 64;
  MST_CUDA_TRY(cudaFuncSetAttribute(strided_attention_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid((unsigned)(seq_len / BQ), (unsigned)heads, (unsigned)batch);
  strided_attention_fwd_kernel<<<grid, ATT_THREADS, smem, (cudaStream_t)stream>>>(tmQ, tmK, tmV, P);
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}
