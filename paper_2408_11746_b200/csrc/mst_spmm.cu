// Row-panel SpMM on the CUDA cores:  out[t, r] = sum_{k in row r} val(k) * in[t, idx[k]].
//
// Forward uses the CSR arrays (r = output feature, idx = input feature); the input gradient uses the CSC view
// (r = input feature, idx = output feature, values fetched through the CSC->CSR permutation), so both are gathers
// with a fixed summation order: no floating-point atomics, run-to-run identical results.
//
// The activations are first copied feature-major once per call (inT[c][t], one coalesced transpose); after that a
// nonzero costs one contiguous read of its column.  A block owns 256 tokens x 120 rows of the output (fewer rows per warp when the grid would not fill the GPU).  A producer
// warp streams [column chunk x 256 tokens] tiles of inT into a ring of shared-memory stages with the TMA unit
// (cp.async.bulk.tensor, this GPU's memory only, no multicast); 15 compute warps each own 8 rows and hold their
// 8 x 256 partial sums in registers (lane = 8 consecutive tokens) across all chunks.  Per nonzero: one warp shuffle
// broadcasts (column, value), one 128-bit shared load fetches the lane's 8 activations, and 8 FMAs accumulate in
// fp32 -- for bf16 layers with the mixed-precision instruction (bf16 x bf16 + fp32), so no unpacking is issued.
// Work is proportional to nnz: a (row, chunk) visit costs a ballot over a 32-entry window of the row kept in
// registers, and global index/value loads happen only when a window is used up (coalesced, 32 entries).
// Rows of unequal nnz: inside a panel the rows are dealt to the warps in order of decreasing nnz, back and forth,
// so every warp gets a similar count; panels are many more than SMs and are scheduled dynamically.  When the longest
// row of the matrix has a thousand entries or more and is far above the mean (recorded on the device when the
// structure changes), a panel keeps a fifth of its row slots free and hands them to its longest rows as extra
// segments (every cnt-th entry of the row each, so that a segment has its share of every column chunk): a long row
// is then summed by up to 1 + 3 x (rows per warp) warps, and the epilogue adds the segments' partial sums in a fixed
// order.
// The output tile leaves through shared memory so that global stores are contiguous along the feature dimension.
#include <cuda.h>

#include "mst_internal.cuh"
#include "mst_tc_gemm.cuh"
#include "mst_tc_ptx.cuh"

namespace {

constexpr int TOK = 256;    // tokens per block (8 per lane)
constexpr int WARPS = 15;   // compute warps; one more warp produces (512 threads: 128 registers each)
constexpr int MAX_RPW = 8;  // rows per warp: 8 (120-row panels) for large outputs, fewer when the grid would not fill the GPU
constexpr int MAX_PANEL = WARPS * MAX_RPW;
constexpr int STAGES = 3;
constexpr int THREADS = (WARPS + 1) * 32;

template <typename T>
struct Cfg;
template <>
struct Cfg<float> {
  static constexpr int KC = 64;   // columns per stage: 64 KiB
  static constexpr int VEC = 4;
};
template <>
struct Cfg<uint16_t> {
  static constexpr int KC = 128;  // 64 KiB
  static constexpr int VEC = 8;
};

__device__ int g_spmm_error = 0;  // sticky: a bounded wait expired

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(uint16_t v) { return __uint_as_float(((uint32_t)v) << 16); }

__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
// fp32 -> bf16, round to nearest even (finite inputs)
__device__ __forceinline__ void store_out(uint16_t* p, float v) {
  uint32_t u = __float_as_uint(v);
  if ((u & 0x7F800000u) != 0x7F800000u) u += 0x7FFFu + ((u >> 16) & 1u);
  *p = (uint16_t)(u >> 16);
}

// acc[0..7] += w * xs[0..7]
__device__ __forceinline__ void fma8(float (&acc)[8], uint32_t wbits, const float* xs) {
  const float w = __uint_as_float(wbits);
  const float4 a = *reinterpret_cast<const float4*>(xs);
  const float4 b = *reinterpret_cast<const float4*>(xs + 4);
  acc[0] = fmaf(w, a.x, acc[0]);
  acc[1] = fmaf(w, a.y, acc[1]);
  acc[2] = fmaf(w, a.z, acc[2]);
  acc[3] = fmaf(w, a.w, acc[3]);
  acc[4] = fmaf(w, b.x, acc[4]);
  acc[5] = fmaf(w, b.y, acc[5]);
  acc[6] = fmaf(w, b.z, acc[6]);
  acc[7] = fmaf(w, b.w, acc[7]);
}
// bf16 operands, fp32 accumulator: d = a * b + c with the exact product (the mixed-precision FMA of sm_100)
__device__ __forceinline__ void fma_bf16(float& acc, uint16_t a, uint16_t b) {
  asm("fma.rn.f32.bf16 %0, %1, %2, %0;" : "+f"(acc) : "h"(a), "h"(b));
}
__device__ __forceinline__ void fma8(float (&acc)[8], uint32_t wbits, const uint16_t* xs) {
  const uint4 v = *reinterpret_cast<const uint4*>(xs);
  const uint16_t w = (uint16_t)wbits;
  const uint32_t xw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint16_t lo, hi;
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(xw[j]));
    fma_bf16(acc[2 * j], w, lo);
    fma_bf16(acc[2 * j + 1], w, hi);
  }
}
// two entries of one row: both operand fetches are issued before the first FMA
__device__ __forceinline__ void fma8x2(float (&acc)[8], uint32_t wa, const float* xa, uint32_t wb, const float* xb) {
  const float4 a0 = *reinterpret_cast<const float4*>(xa), a1 = *reinterpret_cast<const float4*>(xa + 4);
  const float4 b0 = *reinterpret_cast<const float4*>(xb), b1 = *reinterpret_cast<const float4*>(xb + 4);
  const float fa = __uint_as_float(wa), fb = __uint_as_float(wb);
  acc[0] = fmaf(fa, a0.x, acc[0]); acc[1] = fmaf(fa, a0.y, acc[1]); acc[2] = fmaf(fa, a0.z, acc[2]); acc[3] = fmaf(fa, a0.w, acc[3]);
  acc[4] = fmaf(fa, a1.x, acc[4]); acc[5] = fmaf(fa, a1.y, acc[5]); acc[6] = fmaf(fa, a1.z, acc[6]); acc[7] = fmaf(fa, a1.w, acc[7]);
  acc[0] = fmaf(fb, b0.x, acc[0]); acc[1] = fmaf(fb, b0.y, acc[1]); acc[2] = fmaf(fb, b0.z, acc[2]); acc[3] = fmaf(fb, b0.w, acc[3]);
  acc[4] = fmaf(fb, b1.x, acc[4]); acc[5] = fmaf(fb, b1.y, acc[5]); acc[6] = fmaf(fb, b1.z, acc[6]); acc[7] = fmaf(fb, b1.w, acc[7]);
}
__device__ __forceinline__ void fma8x2(float (&acc)[8], uint32_t wa, const uint16_t* xa, uint32_t wb, const uint16_t* xb) {
  const uint4 va = *reinterpret_cast<const uint4*>(xa);
  const uint4 vb = *reinterpret_cast<const uint4*>(xb);
  const uint32_t aw[4] = {va.x, va.y, va.z, va.w}, bw[4] = {vb.x, vb.y, vb.z, vb.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint16_t lo, hi;
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(aw[j]));
    fma_bf16(acc[2 * j], (uint16_t)wa, lo);
    fma_bf16(acc[2 * j + 1], (uint16_t)wa, hi);
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint16_t lo, hi;
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(bw[j]));
    fma_bf16(acc[2 * j], (uint16_t)wb, lo);
    fma_bf16(acc[2 * j + 1], (uint16_t)wb, hi);
  }
}
__device__ __forceinline__ uint32_t weight_bits(float v) { return __float_as_uint(v); }
__device__ __forceinline__ uint32_t weight_bits(uint16_t v) { return (uint32_t)v; }

// inT[c][t] = in[t][c]: 64 x 64 tiles through shared memory, coalesced on both sides.  ldt >= T, multiple of 16 bytes.
template <typename T>
__global__ void __launch_bounds__(256) transpose_in_kernel(const T* __restrict__ in, int64_t ldin, int64_t T_total, int C,
                                                          T* __restrict__ inT, int64_t ldt) {
  __shared__ T tile[64][64 + (sizeof(T) == 2 ? 2 : 1)];
  const int64_t t0 = (int64_t)blockIdx.x * 64;
  const int c0 = blockIdx.y * 64;
  const int x = threadIdx.x & 63, y = threadIdx.x >> 6;   // 4 rows of 64 per pass
#pragma unroll 4
  for (int j = 0; j < 16; ++j) {
    const int tl = y + 4 * j;
    const int64_t t = t0 + tl;
    tile[tl][x] = (t < T_total && c0 + x < C) ? in[t * ldin + c0 + x] : T(0);
  }
  __syncthreads();
#pragma unroll 4
  for (int j = 0; j < 16; ++j) {
    const int cl = y + 4 * j;
    if (c0 + cl < C && t0 + x < ldt) inT[(int64_t)(c0 + cl) * ldt + t0 + x] = tile[x][cl];
  }
}

constexpr int SPLIT_MIN = 64;   // a segment of a split row keeps at least this many entries
constexpr int SPLIT_LONGEST = 1024;   // rows are split only in matrices whose longest row has at least this many

// longest row of the matrix (rows = the ptr array's rows) into *out, which the caller cleared
__global__ void longest_row_kernel(const int32_t* __restrict__ ptr, int R, int32_t* out) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  int v = r < R ? ptr[r + 1] - ptr[r] : 0;
  for (int o = 16; o; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
  if ((threadIdx.x & 31) == 0 && v > 0) atomicMax(out, v);
}

template <typename T, bool PERM, int RPW>
__global__ void __launch_bounds__(THREADS, 1)
spmm_stream_kernel(const __grid_constant__ CUtensorMap tmIn, const int32_t* __restrict__ ptr,
                   const uint16_t* __restrict__ idx, const T* __restrict__ vals, const int32_t* __restrict__ perm,
                   T* __restrict__ out, int64_t ldout, int64_t T_total, int R_total, int C,
                   const int32_t* __restrict__ longest_row) {
  using namespace mst_ptx;
  constexpr int KC = Cfg<T>::KC;
  constexpr int PANEL = WARPS * RPW;          // row slots of a block
  constexpr int SPARE = 3 * RPW;              // slots kept free for extra segments when rows are split
  constexpr int OS_LD = PANEL + 1;
  constexpr uint32_t STAGE_BYTES = (uint32_t)(KC * TOK * sizeof(T));
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 127u) & ~127u;
  unsigned char* tiles = smem_raw + (tiles_base - raw);
  __shared__ uint64_t bars[2 * STAGES];
  __shared__ int nnz_sh[PANEL];               // entries of a slot
  __shared__ int rown_sh[PANEL];              // entries of a row of the panel
  __shared__ int slot_beg[PANEL], slot_end[PANEL];
  __shared__ unsigned char seg_first[PANEL], seg_cnt[PANEL];   // a row's slots: seg_first[row] .. + seg_cnt[row]
  __shared__ unsigned char slot_step[PANEL];  // a slot takes every slot_step-th entry of its row (1: the whole row)
  __shared__ unsigned char order_sh[PANEL];   // order_sh[w * RPW + j] = slot of warp w's j-th row
  __shared__ int abort_sh;
  volatile int* abort_flag = &abort_sh;
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[STAGES]);

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // rows are split when the longest row of the matrix is far above the mean (uniform over the grid; the grid is
  // sized for the split form, whose panels hold fewer rows: without splitting the surplus blocks have nothing to do)
  const int longest = longest_row ? *longest_row : 0;
  // (measured on GPT-2-small shapes with Zipf rows: a gain for rows of thousands of entries, 0.51 -> 0.36 ms on a
  // 768 x 3072 layer; a loss for 768-wide layers, where a fifth more panels cost more than the balance gains)
  const bool split = longest >= SPLIT_LONGEST && (int64_t)longest * R_total > 4 * (int64_t)ptr[R_total] + 64 * (int64_t)R_total;
  const int rows_here = split ? PANEL - SPARE : PANEL;
  const int r0 = blockIdx.x * rows_here;
  if (r0 >= R_total) return;
  const int64_t t0 = (int64_t)blockIdx.y * TOK;
  if (threadIdx.x == 0) {
    abort_sh = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // slots: one per row, or several for the longest rows of the panel when rows are split
  if (threadIdx.x < PANEL) {
    const int r = r0 + threadIdx.x;
    const bool have = (int)threadIdx.x < rows_here && r < R_total;
    rown_sh[threadIdx.x] = have ? ptr[r + 1] - ptr[r] : -1;
    seg_cnt[threadIdx.x] = 1;
    slot_step[threadIdx.x] = 1;
    seg_first[threadIdx.x] = (unsigned char)threadIdx.x;
    nnz_sh[threadIdx.x] = have ? ptr[r + 1] - ptr[r] : -1;
    slot_beg[threadIdx.x] = have ? ptr[r] : 0;
    slot_end[threadIdx.x] = have ? ptr[r + 1] : 0;
  }
  __syncthreads();
  if (split) {   // uniform over the block
    if (warp == 0) {
      // the free slots go, one at a time, to the row whose segments are longest (ties: the lower row)
      int seg[4] = {1, 1, 1, 1};   // rows lane, lane + 32, lane + 64, lane + 96
      for (int it = 0; it < SPARE; ++it) {
        int best = 0, best_row = 0x7FFFFFFF;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int rl = lane + 32 * k;
          if (rl < rows_here) {
            const int n = rown_sh[rl];
            const int per = n > 0 ? (n + seg[k] - 1) / seg[k] : 0;
            if (per > best || (per == best && rl < best_row)) { best = per; best_row = rl; }
          }
        }
        for (int o = 16; o; o >>= 1) {
          const int ob = __shfl_xor_sync(0xffffffffu, best, o), orow = __shfl_xor_sync(0xffffffffu, best_row, o);
          if (ob > best || (ob == best && orow < best_row)) { best = ob; best_row = orow; }
        }
        if (best < 2 * SPLIT_MIN) break;   // uniform: splitting further would leave segments below the minimum
        if ((best_row & 31) == lane) ++seg[best_row >> 5];
      }
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (lane + 32 * k < rows_here) seg_cnt[lane + 32 * k] = (unsigned char)seg[k];
      __syncwarp();
      // first slot of every row: exclusive prefix of the segment counts in row order (lane = four consecutive rows)
      int mine[4], tot = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int rl = lane * 4 + k;
        mine[k] = rl < rows_here ? seg_cnt[rl] : 0;
        tot += mine[k];
      }
      int incl = tot;
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
      }
      int at = incl - tot;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int rl = lane * 4 + k;
        if (rl < rows_here) seg_first[rl] = (unsigned char)at;
        at += mine[k];
      }
      const int used = __shfl_sync(0xffffffffu, incl, 31);
      for (int sl = used + lane; sl < PANEL; sl += 32) {   // slots left over
        nnz_sh[sl] = -1;
        slot_beg[sl] = slot_end[sl] = 0;
        slot_step[sl] = 1;
      }
    }
    __syncthreads();
    if ((int)threadIdx.x < rows_here) {
      const int r = r0 + threadIdx.x;
      // segment j of a row split in cnt takes the entries j, j + cnt, j + 2 cnt, ... of the row: columns still ascend
      // inside a segment, and every segment has its share of every column chunk
      const int n = rown_sh[threadIdx.x], cnt = seg_cnt[threadIdx.x], first = seg_first[threadIdx.x];
      const int beg = n >= 0 ? ptr[r] : 0, end = n >= 0 ? beg + n : 0;
      for (int j = 0; j < cnt; ++j) {
        slot_beg[first + j] = beg + j < end ? beg + j : end;
        slot_end[first + j] = end;
        slot_step[first + j] = (unsigned char)cnt;
        nnz_sh[first + j] = n >= 0 ? (n - j + cnt - 1) / cnt : -1;
      }
    }
    __syncthreads();
  }
  // slots in order of decreasing nnz, dealt to the warps back and forth
  if (threadIdx.x < PANEL) {
    const int mine = nnz_sh[threadIdx.x];
    int rank = 0;
    for (int j = 0; j < PANEL; ++j) {
      const int other = nnz_sh[j];
      rank += (other > mine || (other == mine && j < (int)threadIdx.x)) ? 1 : 0;
    }
    const int round = rank / WARPS, pos = rank % WARPS;
    const int w = (round & 1) ? WARPS - 1 - pos : pos;
    order_sh[w * RPW + round] = (unsigned char)threadIdx.x;
  }
  __syncthreads();
  const int nchunks = (C + KC - 1) / KC;

  if (warp == WARPS) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      for (int c = 0; c < nchunks && !*abort_flag; ++c) {
        if (!mst_ptx::mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag, &g_spmm_error)) break;
        mbar_expect_tx(full0 + 8 * s, STAGE_BYTES);
        tma_load_2d(tiles_base + (uint32_t)s * STAGE_BYTES, &tmIn, (int)t0, c * KC, full0 + 8 * s);
        if (++s == STAGES) { s = 0; ph ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ compute warps
    int rloc[RPW];
    int32_t kwin[RPW], kend[RPW];
    uint32_t wci[RPW], wval[RPW];   // this lane's entry of the row's current 32-entry window: column, value bits
    float acc[RPW][8];
    auto load_window = [&](int rr) {
      const int32_t kk = kwin[rr] + lane * (int)slot_step[rloc[rr]];
      wci[rr] = 0xFFFFFFFFu;
      wval[rr] = 0u;
      if (kk < kend[rr]) {
        wci[rr] = (uint32_t)idx[kk];
        wval[rr] = weight_bits(PERM ? vals[perm[kk]] : vals[kk]);
      }
    };
#pragma unroll
    for (int rr = 0; rr < RPW; ++rr) {
      rloc[rr] = order_sh[warp * RPW + rr];
      kwin[rr] = slot_beg[rloc[rr]];
      kend[rr] = slot_end[rloc[rr]];
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[rr][j] = 0.f;
    }
#pragma unroll
    for (int rr = 0; rr < RPW; ++rr) load_window(rr);

    int s = 0;
    uint32_t ph = 0;
    for (int c = 0; c < nchunks; ++c) {
      if (!mst_ptx::mbar_wait(full0 + 8 * s, ph, abort_flag, &g_spmm_error)) break;
      const T* Xs = reinterpret_cast<const T*>(tiles + (size_t)s * STAGE_BYTES);
      const uint32_t c0 = (uint32_t)(c * KC), c_end = c0 + KC;
#pragma unroll
      for (int rr = 0; rr < RPW; ++rr) {
        while (true) {
          // columns ascend and everything below c0 was consumed in earlier chunks: the entries of this chunk are the
          // lanes whose column lies below c_end and has not been used yet
          const unsigned m = __ballot_sync(0xffffffffu, wci[rr] >= c0 && wci[rr] < c_end);
          if (m == 0) break;
          const int first = __ffs(m) - 1, n = __popc(m);
          // bf16: column and value travel in one shuffle (16 bits each); two entries per trip so that the shared
          // loads of the second overlap the FMAs of the first
          const uint32_t mine = sizeof(T) == 2 ? (((wci[rr] - c0) << 16) | wval[rr]) : 0u;
          int j = first;
          for (; j + 1 < first + n; j += 2) {
            uint32_t ca, wa, cb, wb;
            if (sizeof(T) == 2) {
              const uint32_t pa = __shfl_sync(0xffffffffu, mine, j), pb = __shfl_sync(0xffffffffu, mine, j + 1);
              ca = pa >> 16; wa = pa & 0xFFFFu; cb = pb >> 16; wb = pb & 0xFFFFu;
            } else {
              ca = __shfl_sync(0xffffffffu, wci[rr], j) - c0;
              wa = __shfl_sync(0xffffffffu, wval[rr], j);
              cb = __shfl_sync(0xffffffffu, wci[rr], j + 1) - c0;
              wb = __shfl_sync(0xffffffffu, wval[rr], j + 1);
            }
            fma8x2(acc[rr], wa, Xs + ca * TOK + lane * 8, wb, Xs + cb * TOK + lane * 8);
          }
          if (j < first + n) {
            uint32_t ca, wa;
            if (sizeof(T) == 2) {
              const uint32_t pa = __shfl_sync(0xffffffffu, mine, j);
              ca = pa >> 16; wa = pa & 0xFFFFu;
            } else {
              ca = __shfl_sync(0xffffffffu, wci[rr], j) - c0;
              wa = __shfl_sync(0xffffffffu, wval[rr], j);
            }
            fma8(acc[rr], wa, Xs + ca * TOK + lane * 8);
          }
          if (first + n < 32) break;        // the window still holds entries of later chunks (or the row has ended)
          kwin[rr] += 32 * (int)slot_step[rloc[rr]];   // window used up: next 32 entries of the slot
          load_window(rr);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8 * s);
      if (++s == STAGES) { s = 0; ph ^= 1u; }
    }

    // epilogue: registers -> shared (token-permuted rows, conflict-free) -> global, contiguous along the rows.
    // Named barrier over the compute warps only: every stage has been consumed, the tiles can be overwritten.
    asm volatile("bar.sync 1, %0;" ::"n"(WARPS * 32) : "memory");
    float* Os = reinterpret_cast<float*>(tiles);
#pragma unroll
    for (int rr = 0; rr < RPW; ++rr)
#pragma unroll
      for (int j = 0; j < 8; ++j) Os[(j * 32 + lane) * OS_LD + rloc[rr]] = acc[rr][j];
    asm volatile("bar.sync 1, %0;" ::"n"(WARPS * 32) : "memory");
    if (!split) {
      for (int i = threadIdx.x; i < TOK * PANEL; i += WARPS * 32) {
        const int tt = i / PANEL, rl = i % PANEL;
        const int64_t t = t0 + tt;
        const int r = r0 + rl;
        if (t < T_total && r < R_total) store_out(out + t * ldout + r, Os[((tt & 7) * 32 + (tt >> 3)) * OS_LD + rl]);
      }
    } else {
      constexpr int ROWS = PANEL - SPARE;
      for (int i = threadIdx.x; i < TOK * ROWS; i += WARPS * 32) {
        const int tt = i / ROWS, rl = i % ROWS;
        const int64_t t = t0 + tt;
        const int r = r0 + rl;
        if (t < T_total && r < R_total) {
          const float* o = Os + ((tt & 7) * 32 + (tt >> 3)) * OS_LD + seg_first[rl];
          float v = o[0];
          for (int j = 1; j < (int)seg_cnt[rl]; ++j) v += o[j];   // a split row's segments, in order
          store_out(out + t * ldout + r, v);
        }
      }
    }
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn spmm_encode_fn() {
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

}  // namespace
mst_status_t mst_feature_major_copy(const void* in, int64_t ldin, int64_t T, int C, mst_dtype_t dtype, void* out, int64_t ldt,
                                    cudaStream_t s);
bool mst_feature_major_map(CUtensorMap* tm, const void* base, int64_t T, int C, int64_t ldt, mst_dtype_t dtype, int box_tokens,
                           int box_features);
namespace {

template <typename T>
constexpr size_t spmm_smem() {
  return (size_t)STAGES * Cfg<T>::KC * TOK * sizeof(T) + 128 > (size_t)TOK * (MAX_PANEL + 1) * 4 + 128
             ? (size_t)STAGES * Cfg<T>::KC * TOK * sizeof(T) + 128
             : (size_t)TOK * (MAX_PANEL + 1) * 4 + 128;
}

template <typename T, bool PERM, int RPW>
mst_status_t launch_rpw(const CUtensorMap& tm, const int32_t* ptr, const uint16_t* idx, const void* vals, const int32_t* perm,
                        void* out, int64_t ldout, int64_t T_total, int R_total, int C, const int32_t* longest_row, cudaStream_t s) {
  // with a longest-row record the kernel may split rows: its panels then hold a fifth fewer rows, and the grid is
  // sized for that form
  const int PANEL = longest_row ? WARPS * RPW - 3 * RPW : WARPS * RPW;
  const size_t smem = spmm_smem<T>();
  // per call: the attribute belongs to the current device's copy of the kernel
  MST_CUDA_TRY(cudaFuncSetAttribute(spmm_stream_kernel<T, PERM, RPW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid((unsigned)((R_total + PANEL - 1) / PANEL), (unsigned)((T_total + TOK - 1) / TOK));
  spmm_stream_kernel<T, PERM, RPW><<<grid, THREADS, smem, s>>>(tm, ptr, idx, (const T*)vals, perm, (T*)out, ldout, T_total, R_total, C, longest_row); MST_COUNT_LAUNCH();
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

template <typename T, bool PERM>
mst_status_t launch(const int32_t* ptr, const uint16_t* idx, const void* vals, const int32_t* perm, const void* in,
                    int64_t ldin, void* out, int64_t ldout, int64_t T_total, int R_total, int C, const int32_t* longest_row,
                    cudaStream_t s) {
  // feature-major copy of the activations: [C x ldt], ldt a multiple of 64 tokens
  const int64_t ldt = (T_total + 63) / 64 * 64;
  const mst_dtype_t dt = sizeof(T) == 2 ? MST_BF16 : MST_F32;
  void* inT = nullptr;
  MST_TRY(mst_workspace_kind(MST_WS_COLUMNS, (size_t)C * ldt * sizeof(T), &inT));
  MST_TRY(mst_feature_major_copy(in, ldin, T_total, C, dt, inT, ldt, s));
  CUtensorMap tm;
  if (!mst_feature_major_map(&tm, inT, T_total, C, ldt, dt, TOK, Cfg<T>::KC)) return MST_ERR_SHAPE;
  // rows per warp: the largest panel that still gives every SM a block (small token counts, narrow outputs)
  const int64_t ttiles = (T_total + TOK - 1) / TOK;
  int sms = 148;
  {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
      sms = 148;
  }
  auto blocks = [&](int rpw) { return ((int64_t)R_total + WARPS * rpw - 1) / (WARPS * rpw) * ttiles; };
  if (blocks(8) >= 2 * sms) return launch_rpw<T, PERM, 8>(tm, ptr, idx, vals, perm, out, ldout, T_total, R_total, C, longest_row, s);
  if (blocks(4) >= 2 * sms) return launch_rpw<T, PERM, 4>(tm, ptr, idx, vals, perm, out, ldout, T_total, R_total, C, longest_row, s);
  if (blocks(2) >= sms) return launch_rpw<T, PERM, 2>(tm, ptr, idx, vals, perm, out, ldout, T_total, R_total, C, longest_row, s);
  return launch_rpw<T, PERM, 1>(tm, ptr, idx, vals, perm, out, ldout, T_total, R_total, C, longest_row, s);
}

// Element-wise pass behind the CUDA-core product (the tensor path fuses it into its epilogue instead).
//   GELU:      out = gelu(src) where src = pre if given else out
//   GELU_GRAD: out = out * gelu'(pre)
template <typename T>
__global__ void act_rows_kernel(T* __restrict__ out, int64_t ldout, const T* __restrict__ pre, int64_t ldpre, int64_t rows,
                                int cols, int act) {
  const int64_t n = rows * cols;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t t = e / cols;
    const int c = (int)(e - t * cols);
    T* o = out + t * ldout + c;
    if (act == MST_ACT_GELU) {
      store_out(o, mst_gelu(to_float(*(pre ? pre + t * ldpre + c : o))));
    } else {
      store_out(o, to_float(*o) * mst_gelu_grad(to_float(pre[t * ldpre + c])));
    }
  }
}

template <typename T>
mst_status_t launch_act(void* out, int64_t ldout, const void* pre, int64_t ldpre, int64_t rows, int cols, int act,
                        cudaStream_t s) {
  const int64_t n = rows * cols;
  const int blocks = (int)std::min<int64_t>((n + 255) / 256, 148 * 16);
  act_rows_kernel<T><<<blocks, 256, 0, s>>>((T*)out, ldout, (const T*)pre, ldpre, rows, cols, act); MST_COUNT_LAUNCH();
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

}  // namespace

// feature-major copy out[c][t] = in[t][c] (zero for T <= t < ldt) and its TMA description with a box of
// box_tokens x box_features; shared with the weight-gradient kernel
mst_status_t mst_feature_major_copy(const void* in, int64_t ldin, int64_t T, int C, mst_dtype_t dtype, void* out, int64_t ldt,
                                    cudaStream_t s) {
  dim3 grid((unsigned)(ldt / 64), (unsigned)((C + 63) / 64));
  if (dtype == MST_F32)
    { transpose_in_kernel<float><<<grid, 256, 0, s>>>((const float*)in, ldin, T, C, (float*)out, ldt); MST_COUNT_LAUNCH(); }
  else
    { transpose_in_kernel<uint16_t><<<grid, 256, 0, s>>>((const uint16_t*)in, ldin, T, C, (uint16_t*)out, ldt); MST_COUNT_LAUNCH(); }
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}
bool mst_feature_major_map(CUtensorMap* tm, const void* base, int64_t T, int C, int64_t ldt, mst_dtype_t dtype, int box_tokens,
                           int box_features) {
  EncodeTiledFn enc = spmm_encode_fn();
  if (!enc) return false;
  const size_t es = dtype == MST_F32 ? 4 : 2;
  cuuint64_t dims[2] = {(cuuint64_t)T, (cuuint64_t)C};
  cuuint64_t strides[1] = {(cuuint64_t)ldt * es};
  cuuint32_t box[2] = {(cuuint32_t)box_tokens, (cuuint32_t)box_features};
  cuuint32_t estr[2] = {1u, 1u};
  return enc(tm, dtype == MST_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base),
             dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

mst_status_t mst_spmm_error_flags(int32_t* flags) {
  int v = 0;
  MST_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_spmm_error, sizeof(int)));
  *flags = v;
  return MST_OK;
}

mst_status_t mst_launch_spmm(const mst_layer* L, bool transpose, const void* in, int64_t ldin, int64_t T, void* out,
                             int64_t ldout, cudaStream_t s, int act, void* pre, int64_t ldpre) {
  if (T == 0) return MST_OK;
  const int c = L->cur;
  const int rows = transpose ? L->I : L->O, cols = transpose ? L->O : L->I;
  // Dense-tile tensor-core path: expand W.M to a dense bf16 image [O x I].  Forward: out = in * image^T, the image a
  // K-major operand.  Input gradient: out = in * image, the same image read as an MN-major operand ([K = O] rows of
  // I contiguous columns), so no transposed copy and no CSC view are needed.
  if (act == MST_ACT_NONE && mst_use_sparse_tc_path(L) && mst_sp24_usable(L, transpose ? 1 : 0, in, ldin, out, ldout))
    return mst_sp24_product(const_cast<mst_layer*>(L), transpose ? 1 : 0, in, ldin, T, out, ldout, s);
  if (mst_use_tensor_path(L) && (ldout % 8 == 0) && ((reinterpret_cast<uintptr_t>(out) & 15u) == 0)) {
    // the image is 256-byte aligned by construction: only the activations and the row length decide
    if (mst_tc_gemm_usable(in, ldin, in, L->I)) {
      const uint16_t* image = nullptr;
      MST_TRY(mst_densify(L, s, &image));
      mst_tc_gemm_args a = {};
      a.A = in; a.lda = ldin; a.a_mn_major = 0;
      a.B = image; a.ldb = L->I; a.b_mn_major = transpose ? 1 : 0;
      a.M = T; a.N = rows; a.K = cols;
      a.epilogue = MST_TC_OUT_BF16;
      a.out = out; a.ldc = ldout; a.splits = 1;
      a.act = act; a.pre = pre; a.ldpre = ldpre;
      return mst_tc_gemm(a, s);
    }
  }
  // CUDA cores: the product lands in the pre-activation buffer when the caller keeps one, else in the output
  void* prod = (act == MST_ACT_GELU && pre) ? pre : out;
  const int64_t ldprod = (act == MST_ACT_GELU && pre) ? ldpre : ldout;
  mst_status_t st;
  if (!transpose) {
    // the longest row of the live structure, kept on the device for the kernel's choice between whole and split rows
    int32_t* longest = L->flags + 2;
    if (L->longest_row_version != L->version) {
      MST_CUDA_TRY(cudaMemsetAsync(longest, 0, sizeof(int32_t), s));
      longest_row_kernel<<<(unsigned)((L->O + 255) / 256), 256, 0, s>>>(L->row_ptr[c], L->O, longest); MST_COUNT_LAUNCH();
      MST_CUDA_TRY(cudaGetLastError());
      L->longest_row_version = L->version;
    }
    st = L->dtype == MST_F32
             ? launch<float, false>(L->row_ptr[c], L->col_idx[c], L->vals[c], nullptr, in, ldin, prod, ldprod, T, L->O, L->I, longest, s)
             : launch<uint16_t, false>(L->row_ptr[c], L->col_idx[c], L->vals[c], nullptr, in, ldin, prod, ldprod, T, L->O, L->I, longest, s);
  } else {
    MST_TRY(mst_ensure_csc(L, s));
    st = L->dtype == MST_F32
             ? launch<float, true>(L->col_ptr, L->row_idx, L->vals[c], L->perm, in, ldin, prod, ldprod, T, L->I, L->O, nullptr, s)
             : launch<uint16_t, true>(L->col_ptr, L->row_idx, L->vals[c], L->perm, in, ldin, prod, ldprod, T, L->I, L->O, nullptr, s);
  }
  if (st != MST_OK || act == MST_ACT_NONE) return st;
  return L->dtype == MST_F32 ? launch_act<float>(out, ldout, pre, ldpre, T, rows, act, s)
                             : launch_act<uint16_t>(out, ldout, pre, ldpre, T, rows, act, s);
}

extern "C" mst_status_t mst_spmm_fwd(const mst_layer_t* L, const void* X, int64_t ldx, int64_t T, void* Y, int64_t ldy,
                                     mst_stream_t stream) {
  if (!L || T < 0 || (T > 0 && (!X || !Y))) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  if (ldx < L->I || ldy < L->O) return MST_ERR_SHAPE;
  return mst_launch_spmm(L, false, X, ldx, T, Y, ldy, (cudaStream_t)stream);
}

extern "C" mst_status_t mst_spmm_bwd_x(const mst_layer_t* L, const void* dY, int64_t lddy, int64_t T, void* dX,
                                       int64_t lddx, mst_stream_t stream) {
  if (!L || T < 0 || (T > 0 && (!dY || !dX))) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  if (lddy < L->O || lddx < L->I) return MST_ERR_SHAPE;
  return mst_launch_spmm(L, true, dY, lddy, T, dX, lddx, (cudaStream_t)stream);
}

extern "C" mst_status_t mst_spmm_fwd_gelu(const mst_layer_t* L, const void* X, int64_t ldx, int64_t T, void* Y_pre,
                                          int64_t ldpre, void* H, int64_t ldh, mst_stream_t stream) {
  if (!L || T < 0 || (T > 0 && (!X || !H))) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  if (ldx < L->I || ldh < L->O || (Y_pre && ldpre < L->O)) return MST_ERR_SHAPE;
  return mst_launch_spmm(L, false, X, ldx, T, H, ldh, (cudaStream_t)stream, MST_ACT_GELU, Y_pre, ldpre);
}

extern "C" mst_status_t mst_spmm_bwd_x_gelu(const mst_layer_t* L, const void* dY, int64_t lddy, int64_t T,
                                            const void* Y_pre, int64_t ldpre, void* dPre, int64_t lddpre,
                                            mst_stream_t stream) {
  if (!L || T < 0 || (T > 0 && (!dY || !Y_pre || !dPre))) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  if (lddy < L->O || lddpre < L->I || ldpre < L->I) return MST_ERR_SHAPE;
  return mst_launch_spmm(L, true, dY, lddy, T, dPre, lddpre, (cudaStream_t)stream, MST_ACT_GELU_GRAD,
                         const_cast<void*>(Y_pre), ldpre);
}
