// Device-side building blocks on the 32-bit mask words (shared by the stand-alone structure kernels and by the
// fused topology-update kernel).  In every function one warp handles one word and `lane` is the bit inside it.
#pragma once
#include <stdint.h>

__device__ __forceinline__ unsigned mst_lanemask_lt() {
  unsigned m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

// CSR entries of mask word w.  Source of a value: dense W (pack) or the previous structure (update: an entry present
// before and after keeps its value, a new entry starts at +0).
template <typename V>
__device__ __forceinline__ void mst_fill_csr_word(int64_t w, int lane, const uint32_t* __restrict__ bits,
                                                  const int32_t* __restrict__ wscan, int O, int I, int wpr,
                                                  uint16_t* __restrict__ col_idx, V* __restrict__ vals,
                                                  int32_t* __restrict__ row_ptr, const V* __restrict__ dense_W,
                                                  int64_t ldw, const uint32_t* __restrict__ old_bits,
                                                  const int32_t* __restrict__ old_wscan, const V* __restrict__ old_vals) {
  const int64_t nwords = (int64_t)O * wpr;
  const unsigned wu = (unsigned)w;
  const int o = (int)(wu / (unsigned)wpr), wc = (int)(wu - (unsigned)o * (unsigned)wpr);
  const uint32_t b = bits[w];
  const int32_t base = wscan[w];
  if (wc == 0 && lane == 0) {
    row_ptr[o] = base;
    if (o == O - 1) row_ptr[O] = wscan[nwords];
  }
  if ((b >> lane) & 1u) {
    const int32_t pos = base + __popc(b & mst_lanemask_lt());
    const int c = wc * 32 + lane;
    col_idx[pos] = (uint16_t)c;
    V v;
    if (dense_W) {
      v = dense_W[(int64_t)o * ldw + c];
    } else {
      const uint32_t ob = old_bits[w];
      if ((ob >> lane) & 1u) {
        v = old_vals[old_wscan[w] + __popc(ob & mst_lanemask_lt())];
      } else {
        v = V(0);
      }
    }
    vals[pos] = v;
  }
}

// 32 x 32 bit tile (wr, wc) of the mask -> the same tile of the transposed mask.
__device__ __forceinline__ void mst_transpose_tile(int64_t tile, int lane, const uint32_t* __restrict__ bits, int O, int I,
                                                   int wpr, int wpc, uint32_t* __restrict__ bitsT) {
  const unsigned tu = (unsigned)tile;
  const int wr = (int)(tu / (unsigned)wpr), wc = (int)(tu - (unsigned)wr * (unsigned)wpr);
  const int o = wr * 32 + lane;
  const uint32_t word = o < O ? bits[(int64_t)o * wpr + wc] : 0u;
  uint32_t mine = 0;
#pragma unroll
  for (int c = 0; c < 32; ++c) {
    const uint32_t t = __ballot_sync(0xffffffffu, (word >> c) & 1u);
    if (c == lane) mine = t;
  }
  const int i = wc * 32 + lane;
  if (i < I) bitsT[(int64_t)i * wpc + wr] = mine;
}

// CSC entries of transposed mask word w: row index and the CSR position of the same entry.
__device__ __forceinline__ void mst_fill_csc_word(int64_t w, int lane, const uint32_t* __restrict__ bitsT,
                                                  const int32_t* __restrict__ wscanT, int O, int I, int wpr, int wpc,
                                                  const uint32_t* __restrict__ bits, const int32_t* __restrict__ wscan,
                                                  uint16_t* __restrict__ row_idx, int32_t* __restrict__ perm,
                                                  int32_t* __restrict__ col_ptr) {
  const int64_t nwordsT = (int64_t)I * wpc;
  const unsigned wu = (unsigned)w;
  const int i = (int)(wu / (unsigned)wpc), wr = (int)(wu - (unsigned)i * (unsigned)wpc);
  const uint32_t b = bitsT[w];
  const int32_t base = wscanT[w];
  if (wr == 0 && lane == 0) {
    col_ptr[i] = base;
    if (i == I - 1) col_ptr[I] = wscanT[nwordsT];
  }
  if ((b >> lane) & 1u) {
    const int o = wr * 32 + lane;
    const int32_t posT = base + __popc(b & mst_lanemask_lt());
    const int64_t wf = (int64_t)o * wpr + (i >> 5);
    const uint32_t fb = bits[wf];
    row_idx[posT] = (uint16_t)o;
    perm[posT] = wscan[wf] + __popc(fb & ((1u << (i & 31)) - 1u));
  }
}

// ---- batched forms for kernels where a warp walks many words: B words per trip, loads grouped by dependency level so
// ---- that they overlap (first the mask words and their scans, then the values they point to, then the stores).
template <typename V, int B>
__device__ __forceinline__ void mst_fill_csr_words(int64_t w0, int64_t stride, int64_t w_end, int lane,
                                                   const uint32_t* bits, const int32_t* wscan, int O, int wpr,
                                                   uint16_t* col_idx, V* vals, int32_t* row_ptr,
                                                   const uint32_t* old_bits, const int32_t* old_wscan, const V* old_vals,
                                                   int32_t* max_row) {
  const int64_t nwords = (int64_t)O * wpr;
  uint32_t b[B], ob[B];
  int32_t base[B], obase[B];
#pragma unroll
  for (int j = 0; j < B; ++j) {
    const int64_t w = w0 + j * stride;
    const bool ok = w < w_end;
    b[j] = ok ? bits[w] : 0u;
    base[j] = ok ? wscan[w] : 0;
    ob[j] = ok ? old_bits[w] : 0u;
    obase[j] = ok ? old_wscan[w] : 0;
  }
  V v[B];
#pragma unroll
  for (int j = 0; j < B; ++j) {
    v[j] = V(0);
    if (((b[j] & ob[j]) >> lane) & 1u) v[j] = old_vals[obase[j] + __popc(ob[j] & mst_lanemask_lt())];
  }
#pragma unroll
  for (int j = 0; j < B; ++j) {
    const int64_t w = w0 + j * stride;
    if (w >= w_end) continue;
    const unsigned wu = (unsigned)w;
    const int o = (int)(wu / (unsigned)wpr), wc = (int)(wu - (unsigned)o * (unsigned)wpr);
    if (wc == 0 && lane == 0) {
      row_ptr[o] = base[j];
      if (o == O - 1) row_ptr[O] = wscan[nwords];
      // the next row's first scan entry (or the total) may belong to another block: read only behind a grid barrier,
      // which is what a non-null max_row promises
      if (max_row) atomicMax(max_row, wscan[w + wpr] - base[j]);
    }
    if ((b[j] >> lane) & 1u) {
      const int32_t pos = base[j] + __popc(b[j] & mst_lanemask_lt());
      col_idx[pos] = (uint16_t)(wc * 32 + lane);
      vals[pos] = v[j];
    }
  }
}

template <int B>
__device__ __forceinline__ void mst_fill_csc_words(int64_t w0, int64_t stride, int64_t w_end, int lane,
                                                   const uint32_t* bitsT, const int32_t* wscanT, int I, int wpr, int wpc,
                                                   const uint32_t* bits, const int32_t* wscan, uint16_t* row_idx,
                                                   int32_t* perm, int32_t* col_ptr, int32_t total) {
  uint32_t b[B], fb[B];
  int32_t base[B], fs[B];
  int ii[B], wrr[B];
#pragma unroll
  for (int j = 0; j < B; ++j) {
    const int64_t w = w0 + j * stride;
    const bool ok = w < w_end;
    b[j] = ok ? bitsT[w] : 0u;
    base[j] = ok ? wscanT[w] : 0;
    const unsigned wu = (unsigned)w;
    ii[j] = (int)(wu / (unsigned)wpc);
    wrr[j] = (int)(wu - (unsigned)ii[j] * (unsigned)wpc);
  }
#pragma unroll
  for (int j = 0; j < B; ++j) {
    fb[j] = 0;
    fs[j] = 0;
    if ((b[j] >> lane) & 1u) {
      const int64_t wf = (int64_t)(wrr[j] * 32 + lane) * wpr + (ii[j] >> 5);
      fb[j] = bits[wf];
      fs[j] = wscan[wf];
    }
  }
#pragma unroll
  for (int j = 0; j < B; ++j) {
    const int64_t w = w0 + j * stride;
    if (w >= w_end) continue;
    if (wrr[j] == 0 && lane == 0) {
      col_ptr[ii[j]] = base[j];
      if (ii[j] == I - 1) col_ptr[I] = total;  // the scan's last element, known to every block
    }
    if ((b[j] >> lane) & 1u) {
      const int32_t posT = base[j] + __popc(b[j] & mst_lanemask_lt());
      row_idx[posT] = (uint16_t)(wrr[j] * 32 + lane);
      perm[posT] = fs[j] + __popc(fb[j] & ((1u << (ii[j] & 31)) - 1u));
    }
  }
}
