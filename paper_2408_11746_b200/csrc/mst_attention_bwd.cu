// Strided sparse self-attention, backward (Sec. 3.3): gradients of
//   Out[i] = sum_{j in S_i} P_ij v_j,   P = softmax over S_i of q_i . k_j / sqrt(d),
//   S_i = { j <= i : i - j < l  or  (i - j) mod l == 0 }
// with respect to q, k and v, from the upstream gradient dOut, the forward output and its stored log-sum-exp:
//   delta_i = dOut_i . Out_i                     (= sum_j P_ij dP_ij)
//   P_ij    = exp(q_i . k_j / sqrt(d) - lse_i)   dP_ij = dOut_i . v_j      dS_ij = P_ij (dP_ij - delta_i)
//   dV_j = sum_i P_ij dOut_i      dK_j = sum_i dS_ij q_i / sqrt(d)      dQ_i = sum_j dS_ij k_j / sqrt(d)
//
// Three launches, no atomics (every output element has one owner and a fixed summation order):
//   1. delta: one warp per (token, head).
//   2. dQ, query-centric: a block owns 64 queries of one (sequence, head) and walks the key tiles of their window
//      (stride / 64 + 1 tiles of 64 keys; the tile that starts `stride` positions back also holds the first strided
//      key of every query).  Per tile: S = Q K^T and dP = dOut V^T on the tensor cores (warp-level 16x16x16 bf16
//      fragments, fp32 accumulators), the softmax algebra element-wise on the fp32 tiles in shared memory, then
//      dQ += dS K with dS rounded to bf16.  The strided keys further back (i - 2l, i - 3l, ...: single keys, not
//      tiles) are handled on the CUDA cores.
//   3. dK and dV, key-centric: a block owns 64 keys and walks the query tiles that can see them, with the
//      transposed products (S^T = K Q^T, dP^T = V dOut^T), dV += P^T dOut and dK += dS^T Q; far queries
//      (j + 2l, j + 3l, ...) on the CUDA cores.
// Every warp owns a 16-row strip of each tile, so the element-wise steps need no block-wide barrier; the barriers
// are around the cooperative tile loads only.  Scores, sums and deltas are fp32; P and dS are rounded to bf16 where
// they enter a tensor-core product (as the forward kernel does with P).
#include <cuda_bf16.h>
#include <mma.h>

#include "mst_internal.cuh"
#include "mst_tc_gemm.cuh"

namespace {

using namespace nvcuda;

constexpr int D = 64;        // head dimension
constexpr int TS = 64;       // tile side (queries and keys)
constexpr int BW_THREADS = 256;
constexpr int BW_WARPS = BW_THREADS / 32;
constexpr int LDB = 72;      // row pitch of the bf16 tiles in shared memory (64 + 8: rows 144 bytes apart, no bank aliasing)
constexpr int LDF = 68;      // row pitch of the fp32 tiles
constexpr float SCALE = 0.125f;   // 1 / sqrt(64)

struct BwdParams {
  const __nv_bfloat16 *Q, *K, *V, *Out, *dOut;
  int64_t ld, ldo, lddo;
  const float* lse;    // [batch, heads, seq]
  float* delta;        // [batch, heads, seq]
  __nv_bfloat16 *dQ, *dK, *dV;
  int64_t ldg;
  int batch, seq, heads, stride;
};

__device__ __forceinline__ bool attends(int i, int j, int l) {
  const int back = i - j;
  return back >= 0 && (back < l || back % l == 0);
}

// rows [r0, r0 + 64) of one head's 64 columns -> dst[64][LDB] (row-major, bf16), 16 bytes per thread and step
__device__ __forceinline__ void load_tile(__nv_bfloat16* dst, const __nv_bfloat16* src, int64_t ld, int64_t r0) {
  for (int e = threadIdx.x; e < TS * D / 8; e += BW_THREADS) {
    const int r = e >> 3, c = (e & 7) * 8;
    *reinterpret_cast<uint4*>(dst + r * LDB + c) = *reinterpret_cast<const uint4*>(src + (r0 + r) * ld + c);
  }
}

// the same copy issued asynchronously (cp.async, 16 bytes per request); complete after async_wait_all + a barrier
__device__ __forceinline__ void load_tile_async(__nv_bfloat16* dst, const __nv_bfloat16* src, int64_t ld, int64_t r0) {
  for (int e = threadIdx.x; e < TS * D / 8; e += BW_THREADS) {
    const int r = e >> 3, c = (e & 7) * 8;
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst + r * LDB + c);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src + (r0 + r) * ld + c) : "memory");
  }
}
__device__ __forceinline__ void load_floats_async(float* dst, const float* src, int n) {
  for (int e = threadIdx.x; e < n; e += BW_THREADS) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst + e);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d), "l"(src + e) : "memory");
  }
}
__device__ __forceinline__ void async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

__global__ void attn_delta_kernel(BwdParams P) {
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;   // (token, head)
  const int lane = threadIdx.x & 31;
  const int64_t rows = (int64_t)P.batch * P.seq;
  if (w >= rows * P.heads) return;
  const int64_t t = w / P.heads;
  const int h = (int)(w - t * P.heads);
  const __nv_bfloat162 o = *reinterpret_cast<const __nv_bfloat162*>(P.Out + t * P.ldo + h * D + 2 * lane);
  const __nv_bfloat162 g = *reinterpret_cast<const __nv_bfloat162*>(P.dOut + t * P.lddo + h * D + 2 * lane);
  float s = __bfloat162float(o.x) * __bfloat162float(g.x) + __bfloat162float(o.y) * __bfloat162float(g.y);
  for (int off = 16; off; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
  const int64_t b = t / P.seq;
  const int i = (int)(t - b * P.seq);
  if (lane == 0) P.delta[(b * P.heads + h) * P.seq + i] = s;
}

typedef wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::row_major> FragA;
typedef wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::col_major> FragBt;   // B given as [n][k] rows
typedef wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::row_major> FragB;    // B given as [k][n] rows
typedef wmma::fragment<wmma::accumulator, 16, 16, 16, float> FragC;

// Eight warps per block: warp = (strip of 16 rows, half of the 64 columns).  A warp forms its 16 x 32 part of the two
// score-shaped products, applies the softmax algebra to it, and after a block barrier accumulates its 16 x 32 part of
// the gradient tiles from the complete 16 x 64 strip of weights.

// out [16 x 32] (fp32, pitch LDF) = A strip [16 x 64] * B^T for 32 of B's rows (row n of b_rows holds B^T's column n)
__device__ __forceinline__ void half_abt(float* out, const __nv_bfloat16* a_strip, const __nv_bfloat16* b_rows) {
  FragA a[4];
#pragma unroll
  for (int kb = 0; kb < 4; ++kb) wmma::load_matrix_sync(a[kb], a_strip + kb * 16, LDB);
#pragma unroll
  for (int nb = 0; nb < 2; ++nb) {
    FragC c;
    wmma::fill_fragment(c, 0.f);
#pragma unroll
    for (int kb = 0; kb < 4; ++kb) {
      FragBt b;
      wmma::load_matrix_sync(b, b_rows + nb * 16 * LDB + kb * 16, LDB);
      wmma::mma_sync(c, a[kb], b, c);
    }
    wmma::store_matrix_sync(out + nb * 16, c, LDF, wmma::mem_row_major);
  }
}

// acc[2] (16 x 32, fp32 fragments) += A strip [16 x 64] (bf16) * 32 columns of B [64 x 64] (bf16 rows; b_cols points
// at the first of the 32 columns)
__device__ __forceinline__ void half_ab_acc(FragC (&acc)[2], const __nv_bfloat16* a_strip, const __nv_bfloat16* b_cols) {
#pragma unroll
  for (int kb = 0; kb < 4; ++kb) {
    FragA a;
    wmma::load_matrix_sync(a, a_strip + kb * 16, LDB);
#pragma unroll
    for (int nb = 0; nb < 2; ++nb) {
      FragB b;
      wmma::load_matrix_sync(b, b_cols + kb * 16 * LDB + nb * 16, LDB);
      wmma::mma_sync(acc[nb], a, b, acc[nb]);
    }
  }
}

// ------------------------------------------------------------------------------------------- dQ
__global__ void __launch_bounds__(BW_THREADS) attn_bwd_dq_kernel(BwdParams P) {
  extern __shared__ __align__(128) unsigned char smem[];
  __nv_bfloat16* Qs = reinterpret_cast<__nv_bfloat16*>(smem);   // [64][LDB]
  __nv_bfloat16* Gs = Qs + TS * LDB;                             // dOut tile
  __nv_bfloat16* KV = Gs + TS * LDB;                             // two (K tile, V tile) buffers: the next pair is fetched
  __nv_bfloat16* Sb = KV + 4 * TS * LDB;                         //   while the current one is used
  float* Sf = reinterpret_cast<float*>(Sb + TS * LDB);           // scores, later dQ   [64][LDF]
  float* Pf = Sf + TS * LDF;                                     // dP
  __shared__ float lse_s[TS], del_s[TS];

  const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int q0 = qt * TS, l = P.stride;
  const int64_t row0 = (int64_t)b * P.seq;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t stat0 = ((int64_t)b * P.heads + h) * P.seq;
  load_tile(Qs, P.Q + h * D, P.ld, row0 + q0);
  load_tile(Gs, P.dOut + h * D, P.lddo, row0 + q0);
  if (threadIdx.x < TS) {
    lse_s[threadIdx.x] = P.lse[stat0 + q0 + threadIdx.x];
    del_s[threadIdx.x] = P.delta[stat0 + q0 + threadIdx.x];
  }
  FragC acc[2];
#pragma unroll
  for (int nb = 0; nb < 2; ++nb) wmma::fill_fragment(acc[nb], 0.f);
  const int r_base = (warp & 3) * 16, c_base = (warp >> 2) * 32;
  const int k_first = q0 - l > 0 ? q0 - l : 0;
  load_tile_async(KV, P.K + h * D, P.ld, row0 + k_first);
  load_tile_async(KV + TS * LDB, P.V + h * D, P.ld, row0 + k_first);
  async_commit();
  int buf = 0;
  for (int k0 = k_first; k0 <= q0; k0 += TS, buf ^= 1) {
    async_wait_all();
    __syncthreads();   // this tile has landed for everyone; the other buffer's tile and the weights have been consumed
    const __nv_bfloat16* Ks = KV + buf * 2 * TS * LDB;
    const __nv_bfloat16* Vs = Ks + TS * LDB;
    if (k0 + TS <= q0) {
      load_tile_async(KV + (buf ^ 1) * 2 * TS * LDB, P.K + h * D, P.ld, row0 + k0 + TS);
      load_tile_async(KV + (buf ^ 1) * 2 * TS * LDB + TS * LDB, P.V + h * D, P.ld, row0 + k0 + TS);
      async_commit();
    }
    half_abt(Sf + r_base * LDF + c_base, Qs + r_base * LDB, Ks + c_base * LDB);
    half_abt(Pf + r_base * LDF + c_base, Gs + r_base * LDB, Vs + c_base * LDB);
    __syncwarp();
    // the visited key tiles lie within l + 64 positions behind the queries: a pair is kept iff 0 <= i - j <= l
    // (the window, and the first strided position i - l)
    const int d0 = q0 - k0;
    for (int e = lane; e < 16 * 32; e += 32) {
      const int r = r_base + (e >> 5), c = c_base + (e & 31);
      const int back = d0 + r - c;
      float ds = 0.f;
      if (back >= 0 && back <= l) {
        const float p = __expf(Sf[r * LDF + c] * SCALE - lse_s[r]);
        ds = p * (Pf[r * LDF + c] - del_s[r]);
      }
      Sb[r * LDB + c] = __float2bfloat16(ds);
    }
    __syncthreads();   // the strip of weights is complete (both column halves)
    half_ab_acc(acc, Sb + r_base * LDB, Ks + c_base);
  }
  __syncthreads();     // every warp has read its scores: the array takes dQ now
#pragma unroll
  for (int nb = 0; nb < 2; ++nb)
    wmma::store_matrix_sync(Sf + r_base * LDF + c_base + nb * 16, acc[nb], LDF, wmma::mem_row_major);
  __syncthreads();
  // strided keys beyond the tiles: i - 2l, i - 3l, ...   (lane = two head dimensions)
  for (int r = warp * (TS / BW_WARPS); r < (warp + 1) * (TS / BW_WARPS); ++r) {
    const int i = q0 + r;
    const float2 q = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(Qs + r * LDB + 2 * lane));
    const float2 g = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(Gs + r * LDB + 2 * lane));
    float ax = 0.f, ay = 0.f;
    for (int j = i - 2 * l; j >= 0; j -= l) {
      const float2 k = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(P.K + (row0 + j) * P.ld + h * D + 2 * lane));
      const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(P.V + (row0 + j) * P.ld + h * D + 2 * lane));
      float s = q.x * k.x + q.y * k.y, dp = g.x * v.x + g.y * v.y;
      for (int off = 16; off; off >>= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, off);
        dp += __shfl_xor_sync(0xffffffffu, dp, off);
      }
      const float ds = __expf(s * SCALE - lse_s[r]) * (dp - del_s[r]);
      ax = fmaf(ds, k.x, ax);
      ay = fmaf(ds, k.y, ay);
    }
    const float ox = (Sf[r * LDF + 2 * lane] + ax) * SCALE, oy = (Sf[r * LDF + 2 * lane + 1] + ay) * SCALE;
    *reinterpret_cast<__nv_bfloat162*>(P.dQ + (row0 + i) * P.ldg + h * D + 2 * lane) = __floats2bfloat162_rn(ox, oy);
  }
}

// ------------------------------------------------------------------------------------------- dK, dV
__global__ void __launch_bounds__(BW_THREADS) attn_bwd_dkv_kernel(BwdParams P) {
  extern __shared__ __align__(128) unsigned char smem[];
  __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(smem);
  __nv_bfloat16* Vs = Ks + TS * LDB;
  __nv_bfloat16* QG = Vs + TS * LDB;                             // two (Q tile, dOut tile) buffers
  __nv_bfloat16* Pb = QG + 4 * TS * LDB;                         // P^T, bf16   [key][query]
  __nv_bfloat16* Sb = Pb + TS * LDB;                             // dS^T, bf16
  float* Sf = reinterpret_cast<float*>(Sb + TS * LDB);           // S^T, later dK
  float* Pf = Sf + TS * LDF;                                     // dP^T, later dV
  __shared__ float stat_s[2][2 * TS];   // per buffer: log-sum-exp and delta of the tile's queries

  const int kt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int k0 = kt * TS, l = P.stride;
  const int64_t row0 = (int64_t)b * P.seq;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t stat0 = ((int64_t)b * P.heads + h) * P.seq;
  load_tile(Ks, P.K + h * D, P.ld, row0 + k0);
  load_tile(Vs, P.V + h * D, P.ld, row0 + k0);
  FragC acc_k[2], acc_v[2];
#pragma unroll
  for (int nb = 0; nb < 2; ++nb) {
    wmma::fill_fragment(acc_k[nb], 0.f);
    wmma::fill_fragment(acc_v[nb], 0.f);
  }
  const int r_base = (warp & 3) * 16, c_base = (warp >> 2) * 32;   // this warp's keys, and its half of the columns
  const int q_last = k0 + l < P.seq - TS ? k0 + l : P.seq - TS;
  auto fetch = [&](int q0, int bf) {
    load_tile_async(QG + bf * 2 * TS * LDB, P.Q + h * D, P.ld, row0 + q0);
    load_tile_async(QG + bf * 2 * TS * LDB + TS * LDB, P.dOut + h * D, P.lddo, row0 + q0);
    load_floats_async(stat_s[bf], P.lse + stat0 + q0, TS);
    load_floats_async(stat_s[bf] + TS, P.delta + stat0 + q0, TS);
    async_commit();
  };
  fetch(k0, 0);
  int buf = 0;
  for (int q0 = k0; q0 <= q_last; q0 += TS, buf ^= 1) {
    async_wait_all();
    __syncthreads();   // this query tile has landed for everyone (first trip: also K and V); the other buffer and the
                       // weights of the previous tile have been consumed
    const __nv_bfloat16* Qs = QG + buf * 2 * TS * LDB;
    const __nv_bfloat16* Gs = Qs + TS * LDB;
    const float* lse_s = stat_s[buf];
    const float* del_s = stat_s[buf] + TS;
    if (q0 + TS <= q_last) fetch(q0 + TS, buf ^ 1);
    half_abt(Sf + r_base * LDF + c_base, Ks + r_base * LDB, Qs + c_base * LDB);   // S^T[key][query]
    half_abt(Pf + r_base * LDF + c_base, Vs + r_base * LDB, Gs + c_base * LDB);   // dP^T[key][query]
    __syncwarp();
    const int d0 = q0 - k0;   // the visited query tiles lie within l + 64 positions ahead: kept iff 0 <= i - j <= l
    for (int e = lane; e < 16 * 32; e += 32) {
      const int r = r_base + (e >> 5), c = c_base + (e & 31);      // key r, query c
      const int back = d0 + c - r;
      float p = 0.f, ds = 0.f;
      if (back >= 0 && back <= l) {
        p = __expf(Sf[r * LDF + c] * SCALE - lse_s[c]);
        ds = p * (Pf[r * LDF + c] - del_s[c]);
      }
      Pb[r * LDB + c] = __float2bfloat16(p);
      Sb[r * LDB + c] = __float2bfloat16(ds);
    }
    __syncthreads();   // the strips of weights are complete (both query halves)
    half_ab_acc(acc_v, Pb + r_base * LDB, Gs + c_base);
    half_ab_acc(acc_k, Sb + r_base * LDB, Qs + c_base);
  }
  __syncthreads();     // every warp has read its scores: the arrays take dK and dV now
#pragma unroll
  for (int nb = 0; nb < 2; ++nb) {
    wmma::store_matrix_sync(Sf + r_base * LDF + c_base + nb * 16, acc_k[nb], LDF, wmma::mem_row_major);
    wmma::store_matrix_sync(Pf + r_base * LDF + c_base + nb * 16, acc_v[nb], LDF, wmma::mem_row_major);
  }
  __syncthreads();
  // queries further on that see this key through the stride: j + 2l, j + 3l, ...
  for (int r = warp * (TS / BW_WARPS); r < (warp + 1) * (TS / BW_WARPS); ++r) {
    const int j = k0 + r;
    const float2 k = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(Ks + r * LDB + 2 * lane));
    const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(Vs + r * LDB + 2 * lane));
    float kx = 0.f, ky = 0.f, vx = 0.f, vy = 0.f;
    for (int i = j + 2 * l; i < P.seq; i += l) {
      const float2 q = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(P.Q + (row0 + i) * P.ld + h * D + 2 * lane));
      const float2 g = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(P.dOut + (row0 + i) * P.lddo + h * D + 2 * lane));
      float s = q.x * k.x + q.y * k.y, dp = g.x * v.x + g.y * v.y;
      for (int off = 16; off; off >>= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, off);
        dp += __shfl_xor_sync(0xffffffffu, dp, off);
      }
      const float p = __expf(s * SCALE - P.lse[stat0 + i]);
      const float ds = p * (dp - P.delta[stat0 + i]);
      vx = fmaf(p, g.x, vx);
      vy = fmaf(p, g.y, vy);
      kx = fmaf(ds, q.x, kx);
      ky = fmaf(ds, q.y, ky);
    }
    const int64_t o = (row0 + j) * P.ldg + h * D + 2 * lane;
    *reinterpret_cast<__nv_bfloat162*>(P.dK + o) =
        __floats2bfloat162_rn((Sf[r * LDF + 2 * lane] + kx) * SCALE, (Sf[r * LDF + 2 * lane + 1] + ky) * SCALE);
    *reinterpret_cast<__nv_bfloat162*>(P.dV + o) = __floats2bfloat162_rn(Pf[r * LDF + 2 * lane] + vx, Pf[r * LDF + 2 * lane + 1] + vy);
  }
}

}  // namespace

extern "C" mst_status_t mst_strided_attention_bwd(const void* Q, const void* K, const void* V, int64_t ld, const void* Out,
                                                  int64_t ldo, const void* dOut, int64_t lddo, const float* lse,
                                                  int32_t batch, int32_t seq_len, int32_t heads, int32_t head_dim,
                                                  int32_t stride, void* dQ, void* dK, void* dV, int64_t ldg,
                                                  mst_stream_t stream) {
  if (!Q || !K || !V || !Out || !dOut || !lse || !dQ || !dK || !dV || batch < 0 || seq_len <= 0 || heads <= 0)
    return MST_ERR_INVALID_ARG;
  if (head_dim != D || seq_len % TS != 0 || stride <= 0 || stride % TS != 0) return MST_ERR_SHAPE;
  const int64_t width = (int64_t)heads * D;
  if (ld < width || ldo < width || lddo < width || ldg < width || ld % 8 || ldo % 8 || lddo % 8 || ldg % 8) return MST_ERR_SHAPE;
  if (((reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V) |
        reinterpret_cast<uintptr_t>(Out) | reinterpret_cast<uintptr_t>(dOut) | reinterpret_cast<uintptr_t>(dQ) |
        reinterpret_cast<uintptr_t>(dK) | reinterpret_cast<uintptr_t>(dV)) & 15u) != 0)
    return MST_ERR_SHAPE;
  if (batch == 0) return MST_OK;
  if ((int64_t)batch * seq_len > 0x7FFFFFFF || heads > 65535 || batch > 65535) return MST_ERR_SHAPE;
  cudaStream_t s = (cudaStream_t)stream;
  void* ws = nullptr;
  MST_TRY(mst_workspace_kind(MST_WS_ATTENTION, sizeof(float) * (size_t)batch * heads * seq_len, &ws));
  BwdParams P;
  P.Q = (const __nv_bfloat16*)Q; P.K = (const __nv_bfloat16*)K; P.V = (const __nv_bfloat16*)V;
  P.Out = (const __nv_bfloat16*)Out; P.dOut = (const __nv_bfloat16*)dOut;
  P.ld = ld; P.ldo = ldo; P.lddo = lddo;
  P.lse = lse; P.delta = (float*)ws;
  P.dQ = (__nv_bfloat16*)dQ; P.dK = (__nv_bfloat16*)dK; P.dV = (__nv_bfloat16*)dV;
  P.ldg = ldg;
  P.batch = batch; P.seq = seq_len; P.heads = heads; P.stride = stride;
  const int64_t warps = (int64_t)batch * seq_len * heads;
  attn_delta_kernel<<<(unsigned)((warps * 32 + 255) / 256), 256, 0, s>>>(P); MST_COUNT_LAUNCH();
  const size_t smem_q = (size_t)(7 * TS * LDB) * 2 + (size_t)2 * TS * LDF * 4 + 128;
  const size_t smem_kv = (size_t)(8 * TS * LDB) * 2 + (size_t)2 * TS * LDF * 4 + 128;
  MST_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_dq_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_q));
  MST_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_dkv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_kv));
  dim3 grid((unsigned)(seq_len / TS), (unsigned)heads, (unsigned)batch);
  attn_bwd_dq_kernel<<<grid, BW_THREADS, smem_q, s>>>(P); MST_COUNT_LAUNCH();
  attn_bwd_dkv_kernel<<<grid, BW_THREADS, smem_kv, s>>>(P); MST_COUNT_LAUNCH();
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}
