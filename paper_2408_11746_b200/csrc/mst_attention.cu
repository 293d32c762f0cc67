// Strided sparse self-attention, forward (Sec. 3.3: position i attends to j <= i with i - j < l, and to every l-th
// earlier position j = i - l, i - 2l, ...; every head uses the same pattern).
//
// A tile is (batch, head, 128 queries).  Its window part is two dense tensor-core products on a [128 x (l+128)]
// score tile: the keys q0 - l .. q0 + 127 cover the window of every query of the tile, so there is no loop over key
// blocks and no running softmax.  One persistent block per SM walks over the tiles, its warps specialised:
//   warp 0     TMA producer: Q and the l/128 + 1 key blocks as soon as the previous tile's S = Q K^T has completed,
//              the value blocks as soon as the previous tile's O = P V has completed (single buffers, loads of tile
//              t+1 fly during the softmax of tile t);
//   warp 1     one lane issues tcgen05.mma: S = Q K^T (fp32, tensor memory; two key blocks per instruction), then
//              O = P V key block by key block as the softmax warps announce each block of P;
//   warps 2-9  softmax, two warps per tensor-memory lane quarter (thread = query row, the pair splitting the visible
//              32-key chunks by parity): row maximum (exchanged inside the pair), P = exp(s - max) in bf16 into shared
//              memory in the K-major 128-byte-swizzled operand layout, row sum; the pair's first warp publishes the
//              window's maximum and sum and both go on to the next tile.  Chunks no row of the warp can see are
//              skipped, chunks every row sees in full skip the mask arithmetic.  The position i - l is row r of the
//              tile's first key block, so the mask simply reaches one key further (distance <= l);
//   warps 10-13 the positions outside the tile, i - 2l, i - 3l, ... (at most n/l - 2 per query): a softmax of their
//              own on CUDA cores (scores, maximum, sum, weighted value sum kept in registers), then the tile's
//              epilogue: O from tensor memory once the second product has completed, the two partial softmaxes
//              merged, rows written as bf16 (and the log-sum-exp when asked for).
// Keys before the start of the sequence (q0 < l) are fetched from the rows in front of it (another sequence of the
// batch, or the TMA unit's zero fill before row 0) and masked by position, never by value.
// Every mbarrier wait is bounded (abort flag + sticky error word), as in the contraction kernel.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdlib>
#include <cstring>

#include "mst_internal.cuh"
#include "mst_tc_ptx.cuh"

namespace {

using namespace mst_ptx;

constexpr int D = 64;          // head dimension
constexpr int BQ = 128;        // queries per tile = tensor-memory lanes
constexpr int KB = 128;        // keys per key block
constexpr int TILE_BYTES = 128 * D * 2;  // one [128 x 64] bf16 tile, 16 KiB
constexpr int SM_WARPS = 8;              // softmax warps
constexpr int FAR_WARPS = 4;               // warps for the attended positions outside the tile
constexpr int ATT_THREADS = 64 + 32 * SM_WARPS + 32 * FAR_WARPS;
constexpr int TMEM_COLS = 512;
constexpr int O_COL = 448;     // output accumulator: tensor-memory columns 448..511
constexpr int MAX_FAR = 6;       // attended positions outside the tile, i - 2l, i - 3l, ...: seq / l - 2
constexpr int RED_BYTES = 3 * 2 * BQ * 4;  // a pair's partial row sums, the far positions' (max, sum), a pair's partial maxima

__device__ int g_attn_error = 0;

struct AttnParams {
  const uint16_t *Q, *K, *V;
  int64_t ld;       // elements between consecutive tokens in Q / K / V
  uint16_t* out;
  int64_t ldo;
  float* lse;       // [batch, heads, seq] or NULL
  int seq, heads, stride, batch;
  int nkb;          // key blocks per tile: stride / 128 + 1
  int qblocks;      // seq / 128
  int tiles;        // batch * heads * qblocks
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

// The two warps of a lane quarter meet on an mbarrier of two arrivals (a bounded wait, unlike a named barrier, so an
// aborting block cannot leave a warp behind); shared-memory writes made before it are visible after it.
__device__ __forceinline__ bool pair_meet(uint32_t bar, uint32_t parity, int lane, volatile int* abort_flag) {
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
  return att_wait(bar, parity, abort_flag);
}

// tile index -> (sequence, head, first query); late query blocks first: they carry the most strided positions
__device__ __forceinline__ void tile_coords(const AttnParams& P, int t, int& b, int& h, int& q0) {
  const int qb = P.qblocks - 1 - t / (P.batch * P.heads);
  const int bh = t % (P.batch * P.heads);
  b = bh / P.heads;
  h = bh % P.heads;
  q0 = qb * BQ;
}

// Scores (unscaled) of this warp's 32 rows of tile t against the positions i - 2l, i - 3l, ...:
// se[k] = q_i . k_{i-(k+2)l} for the row i = q0 + qtr*32 + lane.  The warp reads the rows together, eight lanes per
// 128-byte row (four rows per instruction, whole lines), reduces over the eight lanes and hands each row's result to
// the lane that owns the row; one row per lane would touch 32 lines per load instruction.
__device__ __forceinline__ void far_scores(const AttnParams& P, int t, int qtr, int lane, int l, float (&se)[MAX_FAR]) {
  int b, h, q0;
  tile_coords(P, t, b, h, q0);
  const int i_lo = q0 + qtr * 32;
  const int n_far_max = (i_lo + 31) / l - 1 < MAX_FAR ? (i_lo + 31) / l - 1 : MAX_FAR;   // uniform over the warp
  if (n_far_max <= 0) return;
  const int grp = lane >> 3, piece = lane & 7;
  const int64_t tok0 = (int64_t)b * P.seq + i_lo;
  uint4 qv[8];
#pragma unroll
  for (int rr = 0; rr < 8; ++rr)
    qv[rr] = __ldg(reinterpret_cast<const uint4*>(P.Q + (tok0 + rr * 4 + grp) * P.ld + h * D) + piece);
#pragma unroll
  for (int k = 0; k < MAX_FAR; ++k) {
    if (k < n_far_max) {
      // rows of the 32-row group all have the same number of far positions (i_lo and l are multiples of 32)
      float mine = 0.f;
#pragma unroll
      for (int rr = 0; rr < 8; ++rr) {
        const uint4 kv =
            __ldg(reinterpret_cast<const uint4*>(P.K + (tok0 + rr * 4 + grp - (int64_t)(k + 2) * l) * P.ld + h * D) + piece);
        float a = dot8(qv[rr], kv, 0.f);
        a += __shfl_xor_sync(0xffffffffu, a, 1);
        a += __shfl_xor_sync(0xffffffffu, a, 2);
        a += __shfl_xor_sync(0xffffffffu, a, 4);
        const float got = __shfl_sync(0xffffffffu, a, (lane & 3) * 8);   // row rr*4 + (lane & 3)
        if ((lane >> 2) == rr) mine = got;
      }
      se[k] = mine;
    }
  }
}

__global__ void __maxnreg__(128)
strided_attention_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                             const __grid_constant__ CUtensorMap tmV, const AttnParams P) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int nkb = P.nkb;
  const uint32_t q_s = base, k_s = q_s + TILE_BYTES, v_s = k_s + nkb * TILE_BYTES, p_s = v_s + nkb * TILE_BYTES;
  const uint32_t red_s = p_s + 2 * nkb * TILE_BYTES;
  const uint32_t bar0 = red_s + RED_BYTES;
  const uint32_t bar_qk = bar0, bar_v = bar0 + 8, bar_s = bar0 + 16, bar_o = bar0 + 32;
  const uint32_t bar_p0 = bar0 + 88;     // one per key block: P of that block is written (and S read) by all softmax warps
  const uint32_t bar_pair0 = bar0 + 40;  // one per lane quarter
  const uint32_t bar_stat = bar0 + 72, bar_epi = bar0 + 80;  // window statistics published / epilogue of the tile done
  float* red = reinterpret_cast<float*>(smem_raw + (red_s - smem_u32(smem_raw)));  // [2 halves][128 rows]
  __shared__ uint32_t tmem_base_holder;
  __shared__ int abort_sh;
  volatile int* abort_flag = &abort_sh;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int l = P.stride;

  if (threadIdx.x == 0) {
    abort_sh = 0;
    mbar_init(bar_qk, 1);
    mbar_init(bar_v, 1);
    mbar_init(bar_s, 1);
    for (int kb = 0; kb < 3; ++kb) mbar_init(bar_p0 + 8 * kb, SM_WARPS);
    mbar_init(bar_o, 1);
    for (int qq = 0; qq < 4; ++qq) mbar_init(bar_pair0 + 8 * qq, 2);
    mbar_init(bar_stat, SM_WARPS / 2);
    mbar_init(bar_epi, FAR_WARPS);
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

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t it = 0;
      for (int t = blockIdx.x; t < P.tiles && !*abort_flag; t += gridDim.x, ++it) {
        int b, h, q0;
        tile_coords(P, t, b, h, q0);
        const int col = h * D;
        const int row_q = b * P.seq + q0, row_k = row_q - l;
        // Q and K are free once the previous tile's first product has completed, V once its second has
        if (it > 0 && !att_wait(bar_s, (it - 1) & 1u, abort_flag)) break;
        mbar_expect_tx(bar_qk, (uint32_t)((1 + nkb) * TILE_BYTES));
        tma_load_2d(q_s, &tmQ, col, row_q, bar_qk);
        for (int kb = 0; kb < nkb; ++kb) tma_load_2d(k_s + kb * TILE_BYTES, &tmK, col, row_k + kb * KB, bar_qk);
        if (it > 0 && !att_wait(bar_o, (it - 1) & 1u, abort_flag)) break;
        mbar_expect_tx(bar_v, (uint32_t)(nkb * TILE_BYTES));
        for (int kb = 0; kb < nkb; ++kb) tma_load_2d(v_s + kb * TILE_BYTES, &tmV, col, row_k + kb * KB, bar_v);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // S[:, kb*128 .. +128) = Q K_kb^T : M = 128, N = 128, both operands K-major, four K steps of 16
      const uint32_t idesc1 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(KB >> 3) << 17) | ((uint32_t)(BQ >> 4) << 24);
      const uint32_t idesc1_wide = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((2 * KB) >> 3) << 17) | ((uint32_t)(BQ >> 4) << 24);
      // O = P V : M = 128, N = 64, P K-major (64-key blocks of 16 KiB), V as stored (keys x 64: MN-major)
      const uint32_t idesc2 = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(D >> 3) << 17) |
                              ((uint32_t)(BQ >> 4) << 24);
      const uint64_t qd = smem_desc(q_s, 16, 1024), kd0 = smem_desc(k_s, 16, 1024);
      const uint64_t pd0 = smem_desc(p_s, 16, 1024), vd0 = smem_desc(v_s, 8192, 1024);
      uint32_t it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < P.tiles && ok && !*abort_flag; t += gridDim.x, ++it) {
        const uint32_t ph = it & 1u;
        // first product of this tile: S is free (the previous tile's P has been written, so S has been read)
        ok = att_wait(bar_qk, ph, abort_flag);
        if (!ok) break;
        tc_fence_after();
        // key blocks two at a time (N = 256: the blocks are contiguous in shared memory), a last odd one alone:
        // each instruction carries a fixed cost, and the softmax warps wait for the whole of this product
        for (int kb = 0; kb < nkb; kb += 2) {
          const uint64_t kd = kd0 + (uint64_t)(uint32_t)(kb * (TILE_BYTES >> 4));
          const uint32_t idesc = kb + 1 < nkb ? idesc1_wide : idesc1;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            tc_mma(tmem_base + (uint32_t)(kb * KB), qd + (uint64_t)(ks * 2), kd + (uint64_t)(ks * 2), idesc, ks > 0 ? 1u : 0u);
        }
        tc_commit(bar_s);
        // second product, key block by key block as the softmax warps finish writing P for it
        ok = att_wait(bar_v, ph, abort_flag);
        if (ok && it > 0) ok = att_wait(bar_epi, (it - 1) & 1u, abort_flag);   // the previous tile's O has been read
        for (int kb = 0; kb < nkb && ok; ++kb) {
          ok = att_wait(bar_p0 + 8 * kb, ph, abort_flag);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int k8 = 0; k8 < KB / 16; ++k8) {
            const int ks = kb * (KB / 16) + k8;
            const uint64_t pd = pd0 + (uint64_t)(uint32_t)((ks >> 2) * (TILE_BYTES >> 4) + (ks & 3) * 2);
            const uint64_t vd = vd0 + (uint64_t)(uint32_t)(ks * ((16 * 128) >> 4));
            tc_mma(tmem_base + (uint32_t)O_COL, pd, vd, idesc2, ks > 0 ? 1u : 0u);
          }
        }
        if (!ok) break;
        tc_commit(bar_o);
      }
    }
  } else if (warp < 2 + SM_WARPS) {
    // ------------------------------------------------------------------ softmax: thread = query row, two warps per row
    const int q = warp & 3;                 // tensor-memory lane quarter
    const int half = (warp - 2) >> 2;       // which warp of the pair
    const int r = q * 32 + lane;
    const float c = 0.125f * 1.4426950408889634f;  // log2(e) / sqrt(64)
    const uint32_t sw = (uint32_t)(r & 7);
    const int nchunks = nkb * 4;
    float* red_sum = red;                   // [2][128]
    float* red_max = red + 4 * BQ;          // [2][128]
    // The position i - l is row r of the tile's first key block, so its score sits in S and its value in the V tile:
    // the window mask simply reaches one key further (distance <= l).  Positions i - 2l, i - 3l, ... lie outside
    // the tile: the far warps form their softmax partials (maximum, sum, weighted value sum) a tile ahead and the
    // epilogue below merges them with the window's.
    float* win_stat = red + 2 * BQ;         // [128][2]: the window's maximum (unscaled score) and sum, for the epilogue
    int t = blockIdx.x;
    uint32_t it = 0;
    for (; t < P.tiles; t += gridDim.x, ++it) {
      const uint32_t ph = it & 1u;
      int b, h, q0;
      tile_coords(P, t, b, h, q0);
      const int i = q0 + r;                 // position in the sequence
      const int jb = q0 - l;                // first key of the tile (may be negative)
      const int64_t tok = (int64_t)b * P.seq + i;
      float m = -INFINITY;
      const int i_lo = q0 + q * 32, i_hi = i_lo + 31;

      if (!att_wait(bar_s, ph, abort_flag)) break;
      tc_fence_after();
      // The chunks (32 keys) some row of this warp can see are a contiguous range: from the window start of the
      // warp's first row (or key 0) to the diagonal of its last row.
      const int ch_lo = (jb < 0 && -jb / 32 > q) ? -jb / 32 : q;
      const int ch_hi = l / 32 + q;
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
      // pass 1: row maximum over this warp's chunks (those of its parity), the load of the next chunk in flight while
      // this one is reduced; the pair then exchanges its maxima
      {
        auto reduce_max = [&](const uint32_t (&v)[32], int ch) {
          const int j0 = jb + ch * 32;
          float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
          if (j0 >= 0 && j0 + 31 <= i_lo && i_hi - j0 <= l) {            // every row sees the whole chunk
#pragma unroll
            for (int e = 0; e < 32; ++e) m4[e & 3] = fmaxf(m4[e & 3], __uint_as_float(v[e]));
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const int j = j0 + e;
              const bool vis = j >= 0 && j <= i && i - j <= l;
              m4[e & 3] = fmaxf(m4[e & 3], vis ? __uint_as_float(v[e]) : -INFINITY);
            }
          }
          m = fmaxf(fmaxf(m, fmaxf(m4[0], m4[1])), fmaxf(m4[2], m4[3]));
        };
        int ch = ch_lo + ((ch_lo ^ half) & 1);
        if (ch <= ch_hi) {
          uint32_t va[32], vb[32];
          tmem_ld32_nowait(t_row + (uint32_t)(ch * 32), va);
#pragma unroll 1
          while (true) {
            tmem_ld_wait(va);
            if (ch + 2 <= ch_hi) tmem_ld32_nowait(t_row + (uint32_t)((ch + 2) * 32), vb);
            reduce_max(va, ch);
            ch += 2;
            if (ch > ch_hi) break;
            tmem_ld_wait(vb);
            if (ch + 2 <= ch_hi) tmem_ld32_nowait(t_row + (uint32_t)((ch + 2) * 32), va);
            reduce_max(vb, ch);
            ch += 2;
            if (ch > ch_hi) break;
          }
        }
      }
      red_max[half * BQ + r] = m;
      if (!pair_meet(bar_pair0 + 8 * q, 0, lane, abort_flag)) break;   // two meetings per tile: parities 0, 1
      m = fmaxf(m, red_max[(half ^ 1) * BQ + r]);                      // finite: the pair has seen key i itself
      // pass 2 over this warp's chunks (those of its parity): P = exp(s - m) in bf16 into the operand layout,
      // partial row sum in fp32; chunks of its parity outside the visible range are zero-filled
      float s4[4] = {0.f, 0.f, 0.f, 0.f};
      const float mc = m * c;               // finite: key i itself is visible
      {
        auto p_addr = [&](int ch, int g) {
          return p_s + (uint32_t)(ch >> 1) * TILE_BYTES + (uint32_t)r * 128u + (((uint32_t)((ch & 1) * 4 + g) ^ sw) << 4);
        };
#pragma unroll 1
        for (int ch = half; ch < nchunks; ch += 2) {
          if (ch >= ch_lo && ch <= ch_hi) continue;
#pragma unroll
          for (int g = 0; g < 4; ++g)
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(p_addr(ch, g)), "r"(0u) : "memory");
        }
        auto exp_store = [&](const uint32_t (&v)[32], int ch) {
          const int j0 = jb + ch * 32;
          float p[32];
          if (j0 >= 0 && j0 + 31 <= i_lo && i_hi - j0 <= l) {            // every row sees the whole chunk
#pragma unroll
            for (int e = 0; e < 32; ++e) p[e] = ex2_ftz(fmaf(__uint_as_float(v[e]), c, -mc));
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const int j = j0 + e;
              const bool vis = j >= 0 && j <= i && i - j <= l;
              p[e] = vis ? ex2_ftz(fmaf(__uint_as_float(v[e]), c, -mc)) : 0.f;
            }
          }
#pragma unroll
          for (int e = 0; e < 32; ++e) s4[e & 3] += p[e];
          uint32_t w[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) w[e] = pack_bf16(p[2 * e], p[2 * e + 1]);
#pragma unroll
          for (int g = 0; g < 4; ++g)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(p_addr(ch, g)), "r"(w[4 * g]), "r"(w[4 * g + 1]),
                         "r"(w[4 * g + 2]), "r"(w[4 * g + 3])
                         : "memory");
        };
        // visible chunks of this warp's parity, key block by key block; each finished block is announced so that the
        // second product can start on it while the later blocks are still exponentiated
#pragma unroll 1
        for (int kb = 0; kb < nkb; ++kb) {
#pragma unroll 1
          for (int ch = 4 * kb + half; ch < 4 * kb + 4; ch += 2) {
            if (ch < ch_lo || ch > ch_hi) continue;
            uint32_t v[32];
            tmem_ld32(t_row + (uint32_t)(ch * 32), v);
            exp_store(v, ch);
          }
          fence_async_smem();   // P is read by the tensor core through the async proxy
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_p0 + 8 * kb);
        }
      }
      float sum = (s4[0] + s4[1]) + (s4[2] + s4[3]);
      red_sum[half * BQ + r] = sum;
      if (!pair_meet(bar_pair0 + 8 * q, 1, lane, abort_flag)) break;
      sum += red_sum[(half ^ 1) * BQ + r];
      // The epilogue belongs to the far warps: they hold the far positions' partial sums in registers, read O from
      // tensor memory when the second product has completed and write the rows.  The first warp of the pair hands them
      // the window's maximum and sum; these warps go straight on to the next tile.
      if (half == 0) {
        if (it > 0 && !att_wait(bar_epi, (it - 1) & 1u, abort_flag)) break;   // the previous tile's pair has been read
        win_stat[2 * r] = m;
        win_stat[2 * r + 1] = sum;
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_stat);
      }
      tc_fence_before();   // the next tile's products overwrite S and O after this warp's next arrivals
    }
  } else {
    // ------------------------------------------------------------------ far positions: i - 2l, i - 3l, ...
    // A softmax of their own per row (maximum, sum, weighted value sum in fp32, kept in registers), formed while the
    // other warps work on the tile; then the tile's epilogue: O from tensor memory once the second product has
    // completed, the window's maximum and sum from shared memory, the two partial softmaxes merged, rows written.
    const int q = warp & 3;                 // lane quarter = the 32 rows this warp serves
    const int r = q * 32 + lane;
    const float c = 0.125f * 1.4426950408889634f;
    const float* win_stat = red + 2 * BQ;
    const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
    uint32_t it = 0;
    for (int t = blockIdx.x; t < P.tiles; t += gridDim.x, ++it) {
      const uint32_t ph = it & 1u;
      int b, h, q0;
      tile_coords(P, t, b, h, q0);
      const int i = q0 + r;
      const int n_far = i / l - 1 < MAX_FAR ? i / l - 1 : MAX_FAR;   // uniform over the warp; may be <= 0
      float se[MAX_FAR];
      float m_e = -INFINITY, sum_e = 0.f;
      float acc[64];
#pragma unroll
      for (int e = 0; e < 64; ++e) acc[e] = 0.f;
      if (n_far > 0) {
        far_scores(P, t, q, lane, l, se);
#pragma unroll
        for (int k = 0; k < MAX_FAR; ++k) m_e = fmaxf(m_e, k < n_far ? se[k] : -INFINITY);
        const int64_t tok = (int64_t)b * P.seq + i;
#pragma unroll 1
        for (int k = 0; k < n_far; ++k) {
          float sk = se[0];
#pragma unroll
          for (int kk = 1; kk < MAX_FAR; ++kk) sk = kk == k ? se[kk] : sk;
          const float pk = ex2_ftz((sk - m_e) * c);
          sum_e += pk;
          const uint4* vrow = reinterpret_cast<const uint4*>(P.V + (tok - (int64_t)(k + 2) * l) * P.ld + h * D);
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const uint4 x = __ldg(vrow + g);
            acc[8 * g + 0] = fmaf(pk, bf_lo(x.x), acc[8 * g + 0]); acc[8 * g + 1] = fmaf(pk, bf_hi(x.x), acc[8 * g + 1]);
            acc[8 * g + 2] = fmaf(pk, bf_lo(x.y), acc[8 * g + 2]); acc[8 * g + 3] = fmaf(pk, bf_hi(x.y), acc[8 * g + 3]);
            acc[8 * g + 4] = fmaf(pk, bf_lo(x.z), acc[8 * g + 4]); acc[8 * g + 5] = fmaf(pk, bf_hi(x.z), acc[8 * g + 5]);
            acc[8 * g + 6] = fmaf(pk, bf_lo(x.w), acc[8 * g + 6]); acc[8 * g + 7] = fmaf(pk, bf_hi(x.w), acc[8 * g + 7]);
          }
        }
      }
      // epilogue of the tile: O / sum merged with the far positions' partial softmax, written as bf16
      if (!att_wait(bar_o, ph, abort_flag)) break;
      if (!att_wait(bar_stat, ph, abort_flag)) break;
      tc_fence_after();
      {
        const float m_w = win_stat[2 * r];
        float sum = win_stat[2 * r + 1];
        float mm = m_w, a_w = 1.f, a_e = 0.f;
        if (n_far > 0) {
          mm = fmaxf(m_w, m_e);
          a_w = ex2_ftz((m_w - mm) * c);
          a_e = ex2_ftz((m_e - mm) * c);
          sum = fmaf(a_w, sum, a_e * sum_e);
        }
        if (P.lse) P.lse[((int64_t)b * P.heads + h) * P.seq + i] = mm * 0.125f + __logf(sum);
        const float inv = 1.0f / sum;
        uint16_t* orow = P.out + ((int64_t)b * P.seq + i) * P.ldo + h * D;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t v[32];
          tmem_ld32(t_row + (uint32_t)(O_COL + hf * 32), v);
          float o[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = fmaf(a_w, __uint_as_float(v[e]), a_e * acc[hf * 32 + e]) * inv;
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint4 w;
            w.x = pack_bf16(o[8 * g + 0], o[8 * g + 1]);
            w.y = pack_bf16(o[8 * g + 2], o[8 * g + 3]);
            w.z = pack_bf16(o[8 * g + 4], o[8 * g + 5]);
            w.w = pack_bf16(o[8 * g + 6], o[8 * g + 7]);
            reinterpret_cast<uint4*>(orow)[hf * 4 + g] = w;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_epi);
    }
  }

  // ------------------------------------------------------------------ teardown
  if (*abort_flag) {
    for (int t = 0; t < 2000; ++t) __nanosleep(1000);  // let copies and MMAs in flight land
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
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
  if (head_dim != D || seq_len % BQ != 0 || stride <= 0 || stride % 64 != 0) return MST_ERR_SHAPE;
  const int64_t width = (int64_t)heads * D;
  if (ld < width || ldo < width || ld % 8 != 0 || ldo % 8 != 0) return MST_ERR_SHAPE;
  if (((reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V) |
        reinterpret_cast<uintptr_t>(Out)) & 15u) != 0)
    return MST_ERR_SHAPE;
  if (batch == 0) return MST_OK;
  const int64_t rows = (int64_t)batch * seq_len;
  if (rows > 0x7FFFFFFF) return MST_ERR_SHAPE;
  // Two kernels, same results up to rounding order.  The tcgen05 one (whole window scored at once in tensor memory)
  // takes strides 128 and 256 up to 8 strides of sequence; the warp-level one (running softmax over 64-key tiles) takes
  // every stride that is a multiple of 64 and any length.  Measured at 16 x 1024 tokens, 12 heads: stride 256 - 68 us
  // against 72 us, stride 128 - 99 us against 64 us; so the tcgen05 kernel runs where it can at strides from 256 and
  // the warp-level one elsewhere.  MST_ATTN_FWD=tcgen05 / warp forces one of them.
  const bool tm_can = stride % KB == 0 && stride + KB <= O_COL && seq_len / stride - 2 <= MAX_FAR;
  bool tensor_memory_kernel = tm_can && stride >= 256;
  if (const char* e = getenv("MST_ATTN_FWD")) {
    if (strcmp(e, "tcgen05") == 0) {
      if (!tm_can) return MST_ERR_SHAPE;
      tensor_memory_kernel = true;
    } else if (strcmp(e, "warp") == 0) {
      tensor_memory_kernel = false;
    }
  }
  if (!tensor_memory_kernel)
    return mst_attention_fwd_mma(Q, K, V, ld, batch, seq_len, heads, stride, Out, ldo, lse, (cudaStream_t)stream);
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
  P.batch = batch;
  P.qblocks = seq_len / BQ;
  const int64_t tiles = (int64_t)batch * heads * P.qblocks;
  if (tiles > 0x7FFFFFFF) return MST_ERR_SHAPE;
  P.tiles = (int)tiles;
  const size_t smem = (size_t)(1 + 4 * P.nkb) * TILE_BYTES + RED_BYTES + 1024 + 128;
  MST_CUDA_TRY(cudaFuncSetAttribute(strided_attention_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  int dev = 0, sms = 0;
  MST_CUDA_TRY(cudaGetDevice(&dev));
  MST_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int grid = (int)(tiles < sms ? tiles : sms);   // one persistent block per SM
  strided_attention_fwd_kernel<<<grid, ATT_THREADS, smem, (cudaStream_t)stream>>>(tmQ, tmK, tmV, P); MST_COUNT_LAUNCH();
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}
