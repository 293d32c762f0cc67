// Strided sparse self-attention, backward (Sec. 3.3): gradients of
//   Out[i] = sum_{j in S_i} P_ij v_j,   P = softmax over S_i of q_i . k_j / sqrt(d),
//   S_i = { j <= i : i - j < l  or  (i - j) mod l == 0 }
// with respect to q, k and v, from the upstream gradient dOut, the forward output and its stored log-sum-exp:
//   delta_i = dOut_i . Out_i                     (= sum_j P_ij dP_ij)
//   P_ij    = exp(q_i . k_j / sqrt(d) - lse_i)   dP_ij = dOut_i . v_j      dS_ij = P_ij (dP_ij - delta_i)
//   dV_j = sum_i P_ij dOut_i      dK_j = sum_i dS_ij q_i / sqrt(d)      dQ_i = sum_j dS_ij k_j / sqrt(d)
//
// Three launches, no atomics (every output element has one owner and a fixed summation order):
//   1. delta: eight lanes per (token, head) row, 16-byte loads.
//   2. dQ, query-centric: a block owns 64 queries of one (sequence, head) and walks the key tiles of their window
//      (stride / 64 + 1 tiles of 64 keys; the tile that starts `stride` positions back also holds the first strided
//      key of every query).  Per tile: S = Q K^T and dP = dOut V^T on the tensor cores (warp-level mma.sync
//      m16n8k16, bf16 operands fetched with ldmatrix, fp32 accumulators), the softmax algebra on the accumulator
//      registers, then dQ += dS K with dS rounded to bf16 and used as the next A operand straight from the registers
//      (the accumulator layout of two neighbouring 16 x 8 tiles is the A layout).  The strided keys further back (i - 2l, i - 3l, ...) are
//      visited as further tiles of which only the diagonal is kept.
//   3. dK and dV, key-centric: a block owns 64 keys and walks the query tiles that can see them, with the
//      transposed products (S^T = K Q^T, dP^T = V dOut^T), dV += P^T dOut and dK += dS^T Q; far queries
//      (j + 2l, j + 3l, ...) as further tiles, diagonal only.
// Every warp owns a 16-row strip of each tile, so the element-wise steps need no block-wide barrier; the barriers
// are around the cooperative tile loads only.  Scores, sums and deltas are fp32; P and dS are rounded to bf16 where
// they enter a tensor-core product (as the forward kernel does with P).
#include <cuda_bf16.h>

#include "mst_attention_mma.cuh"
#include "mst_internal.cuh"
#include "mst_tc_gemm.cuh"

namespace {
using namespace mst_attn;

struct BwdParams {
  const __nv_bfloat16 *Q, *K, *V, *Out, *dOut;
  int64_t ld, ldo, lddo;
  const float* lse;    // [batch, heads, seq]
  float* delta;        // [batch, heads, seq]
  __nv_bfloat16 *dQ, *dK, *dV;
  int64_t ldg;
  int batch, seq, heads, stride;
};

// delta[b, h, i] = dOut_i . Out_i per head: eight lanes per (token, head) row of 64 elements, 16 bytes per lane and
// tensor, four rows per warp and trip
__global__ void __launch_bounds__(256) attn_delta_kernel(BwdParams P) {
  const int lane = threadIdx.x & 31, grp = lane >> 3, piece = lane & 7;
  const int64_t rows = (int64_t)P.batch * P.seq * P.heads;
  const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t w0 = (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5) * 4; w0 < rows; w0 += warps * 4) {
    const int64_t w = w0 + grp;          // (token, head)
    float s = 0.f;
    int64_t t = 0;
    int h = 0;
    if (w < rows) {
      t = w / P.heads;
      h = (int)(w - t * P.heads);
      const uint4 o = *reinterpret_cast<const uint4*>(P.Out + t * P.ldo + h * D + piece * 8);
      const uint4 g = *reinterpret_cast<const uint4*>(P.dOut + t * P.lddo + h * D + piece * 8);
      const uint32_t ow[4] = {o.x, o.y, o.z, o.w}, gw[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        s = fmaf(__uint_as_float(ow[j] << 16), __uint_as_float(gw[j] << 16), s);
        s = fmaf(__uint_as_float(ow[j] & 0xFFFF0000u), __uint_as_float(gw[j] & 0xFFFF0000u), s);
      }
    }
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    s += __shfl_xor_sync(0xffffffffu, s, 4);
    if (piece == 0 && w < rows) {
      const int64_t b = t / P.seq;
      const int i = (int)(t - b * P.seq);
      P.delta[(b * P.heads + h) * P.seq + i] = s;
    }
  }
}

// ------------------------------------------------------------------------------------------- dQ
__global__ void __launch_bounds__(BW_THREADS, 4) attn_bwd_dq_kernel(BwdParams P) {
  extern __shared__ __align__(128) unsigned char smem[];
  __nv_bfloat16* Qs = reinterpret_cast<__nv_bfloat16*>(smem);   // [64][LDB]
  __nv_bfloat16* Gs = Qs + TS * LDB;                             // dOut tile
  __nv_bfloat16* KV = Gs + TS * LDB;                             // two (K tile, V tile) buffers: the next pair is fetched
  float* Sf = reinterpret_cast<float*>(KV);                      //   while the current one is used; dQ [64][LDF] is staged
                                                                 //   over them when the last tile has been consumed
  __shared__ float lse_s[TS], del_s[TS];

  const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int q0 = qt * TS, l = P.stride;
  const int64_t row0 = (int64_t)b * P.seq;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int64_t stat0 = ((int64_t)b * P.heads + h) * P.seq;
  load_tile_async(Qs, P.Q + h * D, P.ld, row0 + q0);       // all first loads in flight together
  load_tile_async(Gs, P.dOut + h * D, P.lddo, row0 + q0);
  if (threadIdx.x < TS) {
    lse_s[threadIdx.x] = P.lse[stat0 + q0 + threadIdx.x];
    del_s[threadIdx.x] = P.delta[stat0 + q0 + threadIdx.x];
  }
  const int r_base = warp * 16;
  // key tiles: the window's tiles, then one tile per strided position further back (i - 2l, i - 3l, ...), of which
  // only the diagonal (query r, key r) is attended
  const int k_first = q0 - l > 0 ? q0 - l : 0;
  const int n_near = (q0 - k_first) / TS + 1;
  const int n_tiles = n_near + (q0 / l > 1 ? q0 / l - 1 : 0);
  auto tile_start = [&](int ti) { return ti < n_near ? k_first + ti * TS : q0 - (ti - n_near + 2) * l; };
  load_tile_async(KV, P.K + h * D, P.ld, row0 + k_first);
  load_tile_async(KV + TS * LDB, P.V + h * D, P.ld, row0 + k_first);
  async_commit();
  async_wait_all();
  __syncthreads();   // Q, dOut, the statistics and the first key tile are in place
  uint32_t qa[4][4], ga[4][4];
#pragma unroll
  for (int kb = 0; kb < 4; ++kb) {
    load_a(qa[kb], Qs, r_base, kb, lane);
    load_a(ga[kb], Gs, r_base, kb, lane);
  }
  const float nl0 = -lse_s[r_base + g] * 1.4426950408889634f, nl1 = -lse_s[r_base + g + 8] * 1.4426950408889634f;
  const float del0 = del_s[r_base + g], del1 = del_s[r_base + g + 8];
  float acc[8][4];
#pragma unroll
  for (int nb = 0; nb < 8; ++nb) acc[nb][0] = acc[nb][1] = acc[nb][2] = acc[nb][3] = 0.f;
  int buf = 0;
  for (int ti = 0; ti < n_tiles; ++ti, buf ^= 1) {
    const int k0 = tile_start(ti);
    async_wait_all();
    __syncthreads();   // this tile has landed for everyone; the other buffer's tile has been consumed
    const __nv_bfloat16* Ks = KV + buf * 2 * TS * LDB;
    const __nv_bfloat16* Vs = Ks + TS * LDB;
    if (ti + 1 < n_tiles) {
      const int kn = tile_start(ti + 1);
      load_tile_async(KV + (buf ^ 1) * 2 * TS * LDB, P.K + h * D, P.ld, row0 + kn);
      load_tile_async(KV + (buf ^ 1) * 2 * TS * LDB + TS * LDB, P.V + h * D, P.ld, row0 + kn);
      async_commit();
    }
    // a window tile lies within l + 64 positions behind the queries: a pair is kept iff 0 <= i - j <= l (the window,
    // and the first strided position i - l); in a tile further back iff i - j is the tile's own distance
    const int back_lo = ti < n_near ? 0 : q0 - k0, back_hi = ti < n_near ? l : q0 - k0;
    const int back0 = q0 - k0 + r_base + g - 2 * t;   // i - j of this lane's first element of key column 0
    if (ti >= n_near) {
      // a tile further back: query r sees key r of the tile only, so of the 64 keys just the 16 in line with this
      // warp's rows matter (two score tiles of 16 x 8, one 16-key step of the second product)
      const int c0 = r_base;                            // first of those keys
      float sc[2][4], dp[2][4];
#pragma unroll
      for (int nb = 0; nb < 2; ++nb) {
        sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.f;
        dp[nb][0] = dp[nb][1] = dp[nb][2] = dp[nb][3] = 0.f;
      }
      mma_rows_wide<2>(sc, qa, Ks, c0, lane);
      mma_rows_wide<2>(dp, ga, Vs, c0, lane);
#pragma unroll
      for (int nb = 0; nb < 2; ++nb) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          // row r_base + g + 8 (i >> 1) against key c0 + 8 nb + 2 t + (i & 1): kept on the diagonal
          float ds = 0.f;
          if (g + (i >> 1) * 8 == nb * 8 + 2 * t + (i & 1)) {
            const float p = ex2_approx(fmaf(sc[nb][i], SCALE_LOG2E, (i >> 1) ? nl1 : nl0));
            ds = p * (dp[nb][i] - ((i >> 1) ? del1 : del0));
          }
          sc[nb][i] = ds;
        }
      }
      uint32_t a[4];
      a[0] = pack_bf16(sc[0][0], sc[0][1]);
      a[1] = pack_bf16(sc[0][2], sc[0][3]);
      a[2] = pack_bf16(sc[1][0], sc[1][1]);
      a[3] = pack_bf16(sc[1][2], sc[1][3]);
      mma_cols(acc, a, Ks, c0, lane);
      continue;
    }
    // every pair of this warp's rows with the tile's keys is kept: no mask arithmetic (uniform over the warp)
    const bool full = q0 - k0 + r_base - 63 >= back_lo && q0 - k0 + r_base + 15 <= back_hi;
#pragma unroll
    for (int half = 0; half < 2; ++half) {            // 32 keys at a time
      float sc[4][4], dp[4][4];
#pragma unroll
      for (int nb = 0; nb < 4; ++nb) {
        sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.f;
        dp[nb][0] = dp[nb][1] = dp[nb][2] = dp[nb][3] = 0.f;
      }
      mma_rows_wide<4>(sc, qa, Ks, half * 32, lane);
      mma_rows_wide<4>(dp, ga, Vs, half * 32, lane);
      if (full) {
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float p = ex2_approx(fmaf(sc[nb][i], SCALE_LOG2E, (i >> 1) ? nl1 : nl0));
            sc[nb][i] = p * (dp[nb][i] - ((i >> 1) ? del1 : del0));
          }
        }
      } else {
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int back = back0 + (i >> 1) * 8 - (half * 32 + nb * 8 + (i & 1));
            float ds = 0.f;
            if ((unsigned)(back - back_lo) <= (unsigned)(back_hi - back_lo)) {
              const float p = ex2_approx(fmaf(sc[nb][i], SCALE_LOG2E, (i >> 1) ? nl1 : nl0));
              ds = p * (dp[nb][i] - ((i >> 1) ? del1 : del0));
            }
            sc[nb][i] = ds;
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 2; ++j) {                   // 16 keys per step
        uint32_t a[4];
        a[0] = pack_bf16(sc[2 * j][0], sc[2 * j][1]);
        a[1] = pack_bf16(sc[2 * j][2], sc[2 * j][3]);
        a[2] = pack_bf16(sc[2 * j + 1][0], sc[2 * j + 1][1]);
        a[3] = pack_bf16(sc[2 * j + 1][2], sc[2 * j + 1][3]);
        mma_cols(acc, a, Ks, half * 32 + j * 16, lane);
      }
    }
  }
  __syncthreads();   // every warp is done with the key tiles: their storage takes dQ
  store_acc(Sf, acc, r_base, lane);
  __syncwarp();
  for (int r = r_base; r < r_base + 16; ++r) {   // lane = two head dimensions
    const float ox = Sf[r * LDF + 2 * lane] * SCALE, oy = Sf[r * LDF + 2 * lane + 1] * SCALE;
    *reinterpret_cast<__nv_bfloat162*>(P.dQ + (row0 + q0 + r) * P.ldg + h * D + 2 * lane) = __floats2bfloat162_rn(ox, oy);
  }
}

// ------------------------------------------------------------------------------------------- dK, dV
__global__ void __launch_bounds__(BW_THREADS, 3) attn_bwd_dkv_kernel(BwdParams P) {
  extern __shared__ __align__(128) unsigned char smem[];
  __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(smem);
  __nv_bfloat16* Vs = Ks + TS * LDB;
  __nv_bfloat16* QG = Vs + TS * LDB;                             // two (Q tile, dOut tile) buffers
  float* Sf = reinterpret_cast<float*>(QG);                      // dK [64][LDF] and dV are staged over the query buffers
  float* Pf = Sf + TS * LDF;                                     //   when the last tile has been consumed
  __shared__ float stat_s[2][2 * TS];   // per buffer: log-sum-exp and delta of the tile's queries

  const int kt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int k0 = kt * TS, l = P.stride;
  const int64_t row0 = (int64_t)b * P.seq;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int64_t stat0 = ((int64_t)b * P.heads + h) * P.seq;
  load_tile_async(Ks, P.K + h * D, P.ld, row0 + k0);         // all first loads in flight together
  load_tile_async(Vs, P.V + h * D, P.ld, row0 + k0);
  const int r_base = warp * 16;   // this warp's keys
  // query tiles: those whose window reaches these keys, then one tile per strided position further on
  // (j + 2l, j + 3l, ...), of which only the diagonal is attended
  const int q_last = k0 + l < P.seq - TS ? k0 + l : P.seq - TS;
  const int n_near = (q_last - k0) / TS + 1;
  const int m_max = (P.seq - TS - k0) / l;
  const int n_tiles = n_near + (m_max > 1 ? m_max - 1 : 0);
  auto tile_start = [&](int ti) { return ti < n_near ? k0 + ti * TS : k0 + (ti - n_near + 2) * l; };
  auto fetch = [&](int q0, int bf) {
    load_tile_async(QG + bf * 2 * TS * LDB, P.Q + h * D, P.ld, row0 + q0);
    load_tile_async(QG + bf * 2 * TS * LDB + TS * LDB, P.dOut + h * D, P.lddo, row0 + q0);
    load_floats_async(stat_s[bf], P.lse + stat0 + q0, TS);
    load_floats_async(stat_s[bf] + TS, P.delta + stat0 + q0, TS);
    async_commit();
  };
  fetch(k0, 0);
  async_wait_all();
  __syncthreads();   // K, V and the first query tile are in place
  uint32_t ka[4][4], va[4][4];
#pragma unroll
  for (int kb = 0; kb < 4; ++kb) {
    load_a(ka[kb], Ks, r_base, kb, lane);
    load_a(va[kb], Vs, r_base, kb, lane);
  }
  float acc_k[8][4], acc_v[8][4];
#pragma unroll
  for (int nb = 0; nb < 8; ++nb) {
    acc_k[nb][0] = acc_k[nb][1] = acc_k[nb][2] = acc_k[nb][3] = 0.f;
    acc_v[nb][0] = acc_v[nb][1] = acc_v[nb][2] = acc_v[nb][3] = 0.f;
  }
  int buf = 0;
  for (int ti = 0; ti < n_tiles; ++ti, buf ^= 1) {
    const int q0 = tile_start(ti);
    async_wait_all();
    __syncthreads();   // this query tile has landed for everyone; the other buffer has been consumed
    const __nv_bfloat16* Qs = QG + buf * 2 * TS * LDB;
    const __nv_bfloat16* Gs = Qs + TS * LDB;
    const float* lse_s = stat_s[buf];
    const float* del_s = stat_s[buf] + TS;
    if (ti + 1 < n_tiles) fetch(tile_start(ti + 1), buf ^ 1);
    // a window tile lies within l + 64 positions ahead of the keys: a pair is kept iff 0 <= i - j <= l; in a tile
    // further on iff i - j is the tile's own distance
    const int back_lo = ti < n_near ? 0 : q0 - k0, back_hi = ti < n_near ? l : q0 - k0;
    const int back0 = q0 - k0 - (r_base + g) + 2 * t;   // i - j of this lane's first element of query column 0
    if (ti >= n_near) {
      // a tile further on: key r is seen by query r of the tile only, so just the 16 queries in line with this warp's
      // keys matter
      const int c0 = r_base;
      float st[2][4], dp[2][4];
#pragma unroll
      for (int nb = 0; nb < 2; ++nb) {
        st[nb][0] = st[nb][1] = st[nb][2] = st[nb][3] = 0.f;
        dp[nb][0] = dp[nb][1] = dp[nb][2] = dp[nb][3] = 0.f;
      }
      mma_rows_wide<2>(st, ka, Qs, c0, lane);
      mma_rows_wide<2>(dp, va, Gs, c0, lane);
#pragma unroll
      for (int nb = 0; nb < 2; ++nb) {
        const int c = c0 + nb * 8 + 2 * t;
        const float2 ls = *reinterpret_cast<const float2*>(lse_s + c), dl = *reinterpret_cast<const float2*>(del_s + c);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float p = 0.f, ds = 0.f;
          if (g + (i >> 1) * 8 == nb * 8 + 2 * t + (i & 1)) {
            p = ex2_approx(fmaf(st[nb][i], SCALE_LOG2E, -1.4426950408889634f * ((i & 1) ? ls.y : ls.x)));
            ds = p * (dp[nb][i] - ((i & 1) ? dl.y : dl.x));
          }
          st[nb][i] = p;
          dp[nb][i] = ds;
        }
      }
      uint32_t pa[4], da[4];
      pa[0] = pack_bf16(st[0][0], st[0][1]);
      pa[1] = pack_bf16(st[0][2], st[0][3]);
      pa[2] = pack_bf16(st[1][0], st[1][1]);
      pa[3] = pack_bf16(st[1][2], st[1][3]);
      da[0] = pack_bf16(dp[0][0], dp[0][1]);
      da[1] = pack_bf16(dp[0][2], dp[0][3]);
      da[2] = pack_bf16(dp[1][0], dp[1][1]);
      da[3] = pack_bf16(dp[1][2], dp[1][3]);
      mma_cols(acc_v, pa, Gs, c0, lane);
      mma_cols(acc_k, da, Qs, c0, lane);
      continue;
    }
    // every pair of the tile's queries with this warp's keys is kept: no mask arithmetic (uniform over the warp)
    const bool full = q0 - k0 - r_base - 15 >= back_lo && q0 - k0 - r_base + 63 <= back_hi;
#pragma unroll
    for (int half = 0; half < 2; ++half) {              // 32 queries at a time
      float st[4][4], dp[4][4];                         // S^T and dP^T: rows = keys, columns = queries
#pragma unroll
      for (int nb = 0; nb < 4; ++nb) {
        st[nb][0] = st[nb][1] = st[nb][2] = st[nb][3] = 0.f;
        dp[nb][0] = dp[nb][1] = dp[nb][2] = dp[nb][3] = 0.f;
      }
      mma_rows_wide<4>(st, ka, Qs, half * 32, lane);
      mma_rows_wide<4>(dp, va, Gs, half * 32, lane);
#pragma unroll
      for (int nb = 0; nb < 4; ++nb) {
        const int c = half * 32 + nb * 8 + 2 * t;
        float2 ls = *reinterpret_cast<const float2*>(lse_s + c);
        const float2 dl = *reinterpret_cast<const float2*>(del_s + c);
        ls.x *= -1.4426950408889634f;
        ls.y *= -1.4426950408889634f;
        if (full) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float p = ex2_approx(fmaf(st[nb][i], SCALE_LOG2E, (i & 1) ? ls.y : ls.x));
            st[nb][i] = p;
            dp[nb][i] = p * (dp[nb][i] - ((i & 1) ? dl.y : dl.x));
          }
        } else {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int back = back0 + (half * 32 + nb * 8 + (i & 1)) - (i >> 1) * 8;
            float p = 0.f, ds = 0.f;
            if ((unsigned)(back - back_lo) <= (unsigned)(back_hi - back_lo)) {
              p = ex2_approx(fmaf(st[nb][i], SCALE_LOG2E, (i & 1) ? ls.y : ls.x));
              ds = p * (dp[nb][i] - ((i & 1) ? dl.y : dl.x));
            }
            st[nb][i] = p;
            dp[nb][i] = ds;
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 2; ++j) {                     // 16 queries per step
        uint32_t pa[4], da[4];
        pa[0] = pack_bf16(st[2 * j][0], st[2 * j][1]);
        pa[1] = pack_bf16(st[2 * j][2], st[2 * j][3]);
        pa[2] = pack_bf16(st[2 * j + 1][0], st[2 * j + 1][1]);
        pa[3] = pack_bf16(st[2 * j + 1][2], st[2 * j + 1][3]);
        da[0] = pack_bf16(dp[2 * j][0], dp[2 * j][1]);
        da[1] = pack_bf16(dp[2 * j][2], dp[2 * j][3]);
        da[2] = pack_bf16(dp[2 * j + 1][0], dp[2 * j + 1][1]);
        da[3] = pack_bf16(dp[2 * j + 1][2], dp[2 * j + 1][3]);
        mma_cols(acc_v, pa, Gs, half * 32 + j * 16, lane);
        mma_cols(acc_k, da, Qs, half * 32 + j * 16, lane);
      }
    }
  }
  __syncthreads();   // every warp is done with the query tiles: their storage takes dK and dV
  store_acc(Sf, acc_k, r_base, lane);
  store_acc(Pf, acc_v, r_base, lane);
  __syncwarp();
  for (int r = r_base; r < r_base + 16; ++r) {   // lane = two head dimensions
    const int64_t o = (row0 + k0 + r) * P.ldg + h * D + 2 * lane;
    *reinterpret_cast<__nv_bfloat162*>(P.dK + o) = __floats2bfloat162_rn(Sf[r * LDF + 2 * lane] * SCALE, Sf[r * LDF + 2 * lane + 1] * SCALE);
    *reinterpret_cast<__nv_bfloat162*>(P.dV + o) = __floats2bfloat162_rn(Pf[r * LDF + 2 * lane], Pf[r * LDF + 2 * lane + 1]);
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
  const int64_t delta_rows = (int64_t)batch * seq_len * heads;
  const int64_t delta_blocks = (delta_rows / 4 + 7) / 8 + 1;   // eight warps per block, four rows per warp and trip
  attn_delta_kernel<<<(unsigned)(delta_blocks < 148 * 16 ? delta_blocks : 148 * 16), 256, 0, s>>>(P); MST_COUNT_LAUNCH();
  static_assert(2 * TS * LDF * 4 <= 4 * TS * LDB * 2, "the staged gradients must fit the tile buffers");
  const size_t smem_q = (size_t)(6 * TS * LDB) * 2 + 128;
  const size_t smem_kv = (size_t)(6 * TS * LDB) * 2 + 128;
  MST_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_dq_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_q));
  MST_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_dkv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_kv));
  dim3 grid((unsigned)(seq_len / TS), (unsigned)heads, (unsigned)batch);
  attn_bwd_dq_kernel<<<grid, BW_THREADS, smem_q, s>>>(P); MST_COUNT_LAUNCH();
  attn_bwd_dkv_kernel<<<grid, BW_THREADS, smem_kv, s>>>(P); MST_COUNT_LAUNCH();
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}
