// Sparse structure of a layer: bit mask -> CSR (+ CSC view) by popcount, exclusive prefix scan and fill.
//
// The mask is kept as 32-bit words, wpr words per row.  Because canonical CSR order (rows ascending,
// columns ascending) is the order of the flat index o*I+i, the CSR position of an entry is the number of
// set bits before it: an exclusive scan of the per-word popcounts plus a popcount inside the word.
// The same holds for the CSC view on the transposed bit mask.  Everything below is integer work,
// stream-ordered, with no inter-block waiting (the scan is three plain kernels).
#include "mst_internal.cuh"
#include "mst_tc_gemm.cuh"
#include "mst_bits.cuh"

#include <cuda_bf16.h>

namespace {

constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 8;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

__device__ __forceinline__ unsigned lanemask_lt() {
  unsigned m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

// ---- exclusive scan of int32, n up to 2^31: out[0..n], out[n] = total -------------------------
__device__ int block_reduce_sum(int v, int* sh) {
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  int r = 0;
  if (threadIdx.x < 32) {
    r = threadIdx.x < (blockDim.x >> 5) ? sh[threadIdx.x] : 0;
    for (int o = 16; o; o >>= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
  }
  __syncthreads();
  return r;  // valid in warp 0
}

__global__ void scan_tile_sums(const int32_t* __restrict__ in, int64_t n, int32_t* __restrict__ sums,
                               const int* __restrict__ enabled) {
  __shared__ int sh[32];
  if (enabled && !*enabled) return;
  const int64_t base = (int64_t)blockIdx.x * SCAN_TILE;
  int v = 0;
  for (int j = 0; j < SCAN_ITEMS; ++j) {
    const int64_t i = base + (int64_t)j * SCAN_THREADS + threadIdx.x;
    if (i < n) v += in[i];
  }
  const int r = block_reduce_sum(v, sh);
  if (threadIdx.x == 0) sums[blockIdx.x] = r;
}

// one block: in-place exclusive scan of the tile sums (m values)
__global__ void scan_sums_inplace(int32_t* sums, int64_t m, const int* __restrict__ enabled) {
  __shared__ int sh[32];
  __shared__ int carry;
  if (enabled && !*enabled) return;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (int64_t base = 0; base < m; base += blockDim.x) {
    const int64_t i = base + threadIdx.x;
    const int v = i < m ? sums[i] : 0;
    int x = v;  // inclusive scan inside the warp
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, o);
      if ((threadIdx.x & 31) >= o) x += y;
    }
    if ((threadIdx.x & 31) == 31) sh[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x < 32) {
      int w = threadIdx.x < (blockDim.x >> 5) ? sh[threadIdx.x] : 0;
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, w, o);
        if (threadIdx.x >= o) w += y;
      }
      sh[threadIdx.x] = w;  // inclusive over warps
    }
    __syncthreads();
    const int warp_off = (threadIdx.x >> 5) ? sh[(threadIdx.x >> 5) - 1] : 0;
    const int c = carry;
    if (i < m) sums[i] = c + warp_off + x - v;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry = c + warp_off + x;
    __syncthreads();
  }
}

__global__ void scan_tiles(const int32_t* __restrict__ in, int64_t n, const int32_t* __restrict__ sums,
                           int32_t* __restrict__ out, const int* __restrict__ enabled) {
  // thread owns SCAN_ITEMS consecutive elements
  __shared__ int sh[32];
  if (enabled && !*enabled) return;
  const int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
  int v[SCAN_ITEMS];
  int t = 0;
  for (int j = 0; j < SCAN_ITEMS; ++j) {
    v[j] = (base + j < n) ? in[base + j] : 0;
    t += v[j];
  }
  int x = t;
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, x, o);
    if ((threadIdx.x & 31) >= o) x += y;
  }
  if ((threadIdx.x & 31) == 31) sh[threadIdx.x >> 5] = x;
  __syncthreads();
  if (threadIdx.x < 32) {
    int w = threadIdx.x < (SCAN_THREADS >> 5) ? sh[threadIdx.x] : 0;
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, w, o);
      if (threadIdx.x >= o) w += y;
    }
    sh[threadIdx.x] = w;
  }
  __syncthreads();
  int run = sums[blockIdx.x] + ((threadIdx.x >> 5) ? sh[(threadIdx.x >> 5) - 1] : 0) + x - t;
  for (int j = 0; j < SCAN_ITEMS; ++j) {
    if (base + j < n) out[base + j] = run;
    run += v[j];
    if (base + j == n - 1) out[n] = run;
  }
}

__global__ void scan_empty(int32_t* out) { out[0] = 0; }

// ---- bit mask construction ---------------------------------------------------------------------
// one warp per mask word: lane = column inside the word
__global__ void mask_bytes_to_bits(const uint8_t* __restrict__ mask, int O, int I, int wpr, uint32_t* __restrict__ bits) {
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= (int64_t)O * wpr) return;
  const int o = (int)(w / wpr), c = (int)(w % wpr) * 32 + lane;
  const bool on = c < I && mask[(int64_t)o * I + c] != 0;
  const unsigned b = __ballot_sync(0xffffffffu, on);
  if (lane == 0) bits[w] = b;
}

__global__ void popc_words(const uint32_t* __restrict__ bits, int64_t n, int32_t* __restrict__ cnt) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) cnt[i] = __popc(bits[i]);
}

// new = (old & ~pruned) | grad | rand
__global__ void combine_bits(const uint32_t* __restrict__ oldb, const uint32_t* __restrict__ pruned,
                             const uint32_t* __restrict__ grad, const uint32_t* __restrict__ rnd, int64_t n,
                             uint32_t* __restrict__ out, int32_t* __restrict__ cnt) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    const uint32_t b = (oldb[i] & ~pruned[i]) | grad[i] | rnd[i];
    out[i] = b;
    cnt[i] = __popc(b);
  }
}

// ---- CSR fill: one warp per word, lane = bit ---------------------------------------------------
// Source of a value: dense W (pack) or the previous structure (update: survivors keep their value, others +0).
template <typename V>
__global__ void fill_csr(const uint32_t* __restrict__ bits, const int32_t* __restrict__ wscan, int O, int I, int wpr,
                         uint16_t* __restrict__ col_idx, V* __restrict__ vals, int32_t* __restrict__ row_ptr,
                         const V* __restrict__ dense_W, int64_t ldw, const uint32_t* __restrict__ old_bits,
                         const int32_t* __restrict__ old_wscan, const V* __restrict__ old_vals) {
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (w >= (int64_t)O * wpr) return;
  mst_fill_csr_word<V>(w, threadIdx.x & 31, bits, wscan, O, I, wpr, col_idx, vals, row_ptr, dense_W, ldw, old_bits,
                       old_wscan, old_vals);
}

// ---- bit transpose: one warp per 32x32 bit tile -------------------------------------------------
__global__ void transpose_bits(const uint32_t* __restrict__ bits, int O, int I, int wpr, int wpc,
                               uint32_t* __restrict__ bitsT) {
  const int64_t tile = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (tile >= (int64_t)wpc * wpr) return;
  mst_transpose_tile(tile, threadIdx.x & 31, bits, O, I, wpr, wpc, bitsT);
}

__global__ void fill_csc(const uint32_t* __restrict__ bitsT, const int32_t* __restrict__ wscanT, int O, int I, int wpr,
                         int wpc, const uint32_t* __restrict__ bits, const int32_t* __restrict__ wscan,
                         uint16_t* __restrict__ row_idx, int32_t* __restrict__ perm, int32_t* __restrict__ col_ptr) {
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (w >= (int64_t)I * wpc) return;
  mst_fill_csc_word(w, threadIdx.x & 31, bitsT, wscanT, O, I, wpr, wpc, bits, wscan, row_idx, perm, col_ptr);
}

// ---- dense bf16 image of W.M (or its transpose) for the tensor-core path ----------------------------------------------
// One thread per 8 consecutive columns: the stored values of those columns are consecutive in CSR (or CSC) order, so
// the thread reads them in one run and writes one 16-byte vector (value or +0 per column).  Every element is written,
// no separate clear.  Needs C % 8 == 0 (the tensor-core path requires it anyway).
__global__ void densify_from_bits(const uint32_t* __restrict__ bits, const int32_t* __restrict__ wscan, int R, int C,
                                  int wpr, const uint16_t* __restrict__ vals, const int32_t* __restrict__ perm,
                                  uint16_t* __restrict__ dense) {
  mst_grid_launch_dependents();
  mst_grid_dependency_wait();
  const unsigned g = blockIdx.x * blockDim.x + threadIdx.x;  // group of 8 columns
  const unsigned gpr = (unsigned)C >> 3;                     // groups per row
  if (g >= (unsigned)R * gpr) return;
  const unsigned r = g / gpr, c8 = g - r * gpr;
  const unsigned w = r * (unsigned)wpr + (c8 >> 2);
  const uint32_t word = bits[w];
  const unsigned sh = (c8 & 3u) * 8u;
  uint32_t m = (word >> sh) & 0xFFu;
  uint16_t out[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  if (m) {
    int32_t pos = wscan[w] + __popc(word & ((1u << sh) - 1u));
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if ((m >> j) & 1u) {
        out[j] = vals[perm ? perm[pos] : pos];
        ++pos;
      }
    }
  }
  uint4 v;
  v.x = (uint32_t)out[0] | ((uint32_t)out[1] << 16);
  v.y = (uint32_t)out[2] | ((uint32_t)out[3] << 16);
  v.z = (uint32_t)out[4] | ((uint32_t)out[5] << 16);
  v.w = (uint32_t)out[6] | ((uint32_t)out[7] << 16);
  *reinterpret_cast<uint4*>(dense + (size_t)r * C + (size_t)c8 * 8) = v;
}

// ---- export / validate ---------------------------------------------------------------------------
__global__ void widen_u16(const uint16_t* __restrict__ in, int64_t n, int32_t* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = in[i];
}

__global__ void validate_rows(const int32_t* __restrict__ row_ptr, const uint16_t* __restrict__ col_idx,
                              const uint32_t* __restrict__ bits, int O, int I, int wpr, int64_t nnz,
                              int32_t* __restrict__ flags) {
  const int o = blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= O) return;
  bool bad = false;
  const int32_t a = row_ptr[o], b = row_ptr[o + 1];
  if (o == 0 && a != 0) bad = true;
  if (o == O - 1 && b != nnz) bad = true;
  if (a > b || a < 0 || b > nnz) {
    bad = true;
  } else {
    int prev = -1, pc = 0;
    for (int32_t k = a; k < b; ++k) {
      const int c = col_idx[k];
      if (c <= prev || c >= I) { bad = true; break; }
      if (!((bits[(int64_t)o * wpr + (c >> 5)] >> (c & 31)) & 1u)) { bad = true; break; }
      prev = c;
    }
    for (int w = 0; w < wpr; ++w) pc += __popc(bits[(int64_t)o * wpr + w]);
    if (pc != b - a) bad = true;
  }
  if (bad) atomicOr(&flags[0], MST_FLAG_CORRUPT);
}

__global__ void validate_cols(const int32_t* __restrict__ col_ptr, const uint16_t* __restrict__ row_idx,
                              const int32_t* __restrict__ perm, const int32_t* __restrict__ row_ptr,
                              const uint16_t* __restrict__ col_idx, int O, int I, int64_t nnz,
                              int32_t* __restrict__ flags) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= I) return;
  bool bad = false;
  const int32_t a = col_ptr[i], b = col_ptr[i + 1];
  if (i == 0 && a != 0) bad = true;
  if (i == I - 1 && b != nnz) bad = true;
  if (a > b || a < 0 || b > nnz) {
    bad = true;
  } else {
    int prev = -1;
    for (int32_t k = a; k < b; ++k) {
      const int o = row_idx[k];
      const int32_t p = perm[k];
      if (o <= prev || o >= O || p < 0 || p >= nnz) { bad = true; break; }
      if (p < row_ptr[o] || p >= row_ptr[o + 1] || col_idx[p] != i) { bad = true; break; }
      prev = o;
    }
  }
  if (bad) atomicOr(&flags[0], MST_FLAG_CORRUPT);
}

inline unsigned blocks_for(int64_t n, int per_block) { return (unsigned)((n + per_block - 1) / per_block); }

}  // namespace

int64_t mst_scan_block_sums_len(int64_t n) { return (n + SCAN_TILE - 1) / SCAN_TILE + 1 + 1024; }

mst_status_t mst_scan_i32_if(const int32_t* in, int32_t* out, int64_t n, int32_t* block_sums, const int* enabled,
                             cudaStream_t s) {
  if (n <= 0) {
    scan_empty<<<1, 1, 0, s>>>(out); MST_COUNT_LAUNCH();
    MST_CUDA_TRY(cudaGetLastError());
    return MST_OK;
  }
  const int64_t tiles = (n + SCAN_TILE - 1) / SCAN_TILE;
  scan_tile_sums<<<(unsigned)tiles, SCAN_THREADS, 0, s>>>(in, n, block_sums, enabled); MST_COUNT_LAUNCH();
  scan_sums_inplace<<<1, 1024, 0, s>>>(block_sums, tiles, enabled); MST_COUNT_LAUNCH();
  scan_tiles<<<(unsigned)tiles, SCAN_THREADS, 0, s>>>(in, n, block_sums, out, enabled); MST_COUNT_LAUNCH();
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

mst_status_t mst_scan_i32(const int32_t* in, int32_t* out, int64_t n, int32_t* block_sums, cudaStream_t s) {
  return mst_scan_i32_if(in, out, n, block_sums, nullptr, s);
}

// bits[set] must be final.  Computes wscan[set], row_ptr[set], col_idx[set], vals[set].
mst_status_t mst_rebuild_from_bits(mst_layer* L, int set, const void* dense_W, int64_t ldw, int old_set,
                                   cudaStream_t s) {
  popc_words<<<blocks_for(L->nwords, 256), 256, 0, s>>>(L->bits[set], L->nwords, L->word_cnt); MST_COUNT_LAUNCH();
  MST_TRY(mst_scan_i32(L->word_cnt, L->wscan[set], L->nwords, L->block_sums, s));
  const unsigned grid = blocks_for(L->nwords * 32, 256);
  if (L->dtype == MST_F32) {
    fill_csr<float><<<grid, 256, 0, s>>>(L->bits[set], L->wscan[set], L->O, L->I, L->wpr, L->col_idx[set],
                                         (float*)L->vals[set], L->row_ptr[set], (const float*)dense_W, ldw,
                                         L->bits[old_set], L->wscan[old_set], (const float*)L->vals[old_set]); MST_COUNT_LAUNCH();
  } else {
    fill_csr<uint16_t><<<grid, 256, 0, s>>>(L->bits[set], L->wscan[set], L->O, L->I, L->wpr, L->col_idx[set],
                                            (uint16_t*)L->vals[set], L->row_ptr[set], (const uint16_t*)dense_W, ldw,
                                            L->bits[old_set], L->wscan[old_set], (const uint16_t*)L->vals[old_set]); MST_COUNT_LAUNCH();
  }
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

// CSC view of the live set.
mst_status_t mst_build_csc(mst_layer* L, cudaStream_t s) {
  MST_TRY(mst_alloc_csc(L));
  const int c = L->cur;
  transpose_bits<<<blocks_for((int64_t)L->wpc * L->wpr * 32, 256), 256, 0, s>>>(L->bits[c], L->O, L->I, L->wpr, L->wpc,
                                                                                L->bitsT); MST_COUNT_LAUNCH();
  popc_words<<<blocks_for(L->nwordsT, 256), 256, 0, s>>>(L->bitsT, L->nwordsT, L->word_cnt); MST_COUNT_LAUNCH();
  MST_TRY(mst_scan_i32(L->word_cnt, L->wscanT, L->nwordsT, L->block_sums, s));
  fill_csc<<<blocks_for(L->nwordsT * 32, 256), 256, 0, s>>>(L->bitsT, L->wscanT, L->O, L->I, L->wpr, L->wpc, L->bits[c],
                                                            L->wscan[c], L->row_idx, L->perm, L->col_ptr); MST_COUNT_LAUNCH();
  MST_CUDA_TRY(cudaGetLastError());
  L->csc_valid = 1;
  return MST_OK;
}

mst_status_t mst_ensure_csc(const mst_layer* L, cudaStream_t s) {
  if (L->csc_valid) return MST_OK;
  return mst_build_csc(const_cast<mst_layer*>(L), s);
}

// Dense bf16 image of W.M for the dense-tile kernels.  Without value tracking the image is rebuilt at every call
// anyway, so it lives in a per-device scratch buffer shared by all layers (no per-layer memory; like the other
// scratch kinds, calls that use it must not overlap on the GPU).  With value tracking the layer keeps its own image
// and reuses it until the mask or the values change.
mst_status_t mst_densify(const mst_layer* L, cudaStream_t s, const uint16_t** image) {
  const int c = L->cur;
  if (L->nnz == L->N) {  // every entry kept: the CSR values in row-major order are the dense matrix
    *image = (const uint16_t*)L->vals[c];
    return MST_OK;
  }
  uint16_t* dst = nullptr;
  if (L->track_values) {
    MST_TRY(mst_alloc_dense(const_cast<mst_layer*>(L)));
    dst = L->dense_w;
    *image = dst;
    if (L->dense_version == L->version && L->dense_epoch == L->values_epoch) return MST_OK;
    L->dense_version = L->version;
    L->dense_epoch = L->values_epoch;
  } else {
    void* ws = nullptr;
    MST_TRY(mst_workspace_kind(MST_WS_IMAGE, 2 * (size_t)L->N, &ws));
    dst = (uint16_t*)ws;
    *image = dst;
  }
  const int64_t groups = L->N / 8;  // callers guarantee I % 8 == 0
  MST_CUDA_TRY(mst_launch_overlapped(densify_from_bits, dim3(blocks_for(groups, 256)), dim3(256), 0, s,
                                     (const uint32_t*)L->bits[c], (const int32_t*)L->wscan[c], L->O, L->I, L->wpr,
                                     (const uint16_t*)L->vals[c], (const int32_t*)nullptr, dst));
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

// new mask of an update from the three selection results; leaves popcounts in word_cnt
mst_status_t mst_combine_update_bits(mst_layer* L, int new_set, cudaStream_t s) {
  combine_bits<<<blocks_for(L->nwords, 256), 256, 0, s>>>(L->bits[L->cur], L->pruned_bits, L->grad_bits, L->rand_bits,
                                                          L->nwords, L->bits[new_set], L->word_cnt); MST_COUNT_LAUNCH();
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

extern "C" mst_status_t mst_pack(mst_layer_t* L, const void* W_dense, int64_t ldw, const uint8_t* mask,
                                 mst_stream_t stream) {
  if (!L || !W_dense || !mask) return MST_ERR_INVALID_ARG;
  if (ldw < L->I) return MST_ERR_SHAPE;
  cudaStream_t s = (cudaStream_t)stream;
  const int set = L->cur;
  L->nnz = -1;
  mask_bytes_to_bits<<<blocks_for(L->nwords * 32, 256), 256, 0, s>>>(mask, L->O, L->I, L->wpr, L->bits[set]); MST_COUNT_LAUNCH();
  popc_words<<<blocks_for(L->nwords, 256), 256, 0, s>>>(L->bits[set], L->nwords, L->word_cnt); MST_COUNT_LAUNCH();
  MST_TRY(mst_scan_i32(L->word_cnt, L->wscan[set], L->nwords, L->block_sums, s));
  int32_t total = 0;
  MST_CUDA_TRY(cudaMemcpyAsync(&total, L->wscan[set] + L->nwords, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  MST_CUDA_TRY(cudaStreamSynchronize(s));
  if (total > L->cap) return MST_ERR_CAPACITY;
  MST_TRY(mst_rebuild_from_bits(L, set, W_dense, ldw, set, s));
  L->nnz = total;
  ++L->version;
  // the CSC view serves the CUDA-core input gradient, the CSC export and the structure check: layers on the tensor
  // path get it on demand
  if (mst_use_tensor_path(L)) L->csc_valid = 0;
  else MST_TRY(mst_build_csc(L, s));
  MST_CUDA_TRY(cudaStreamSynchronize(s));
  return MST_OK;
}

extern "C" mst_status_t mst_export_csr(const mst_layer_t* L, int32_t* row_ptr, int32_t* col_idx, void* vals,
                                       mst_stream_t stream) {
  if (!L) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  cudaStream_t s = (cudaStream_t)stream;
  const int c = L->cur;
  if (row_ptr)
    MST_CUDA_TRY(cudaMemcpyAsync(row_ptr, L->row_ptr[c], sizeof(int32_t) * (L->O + 1), cudaMemcpyDeviceToDevice, s));
  if (col_idx && L->nnz > 0) { widen_u16<<<blocks_for(L->nnz, 256), 256, 0, s>>>(L->col_idx[c], L->nnz, col_idx); MST_COUNT_LAUNCH(); }
  if (vals && L->nnz > 0)
    MST_CUDA_TRY(cudaMemcpyAsync(vals, L->vals[c], mst_elem_size(L->dtype) * L->nnz, cudaMemcpyDeviceToDevice, s));
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

extern "C" mst_status_t mst_export_csc(const mst_layer_t* L, int32_t* col_ptr, int32_t* row_idx, int32_t* perm,
                                       mst_stream_t stream) {
  if (!L) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  cudaStream_t s = (cudaStream_t)stream;
  MST_TRY(mst_ensure_csc(L, s));
  if (col_ptr)
    MST_CUDA_TRY(cudaMemcpyAsync(col_ptr, L->col_ptr, sizeof(int32_t) * (L->I + 1), cudaMemcpyDeviceToDevice, s));
  if (row_idx && L->nnz > 0) { widen_u16<<<blocks_for(L->nnz, 256), 256, 0, s>>>(L->row_idx, L->nnz, row_idx); MST_COUNT_LAUNCH(); }
  if (perm && L->nnz > 0)
    MST_CUDA_TRY(cudaMemcpyAsync(perm, L->perm, sizeof(int32_t) * L->nnz, cudaMemcpyDeviceToDevice, s));
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

extern "C" mst_status_t mst_validate(const mst_layer_t* L, mst_stream_t stream) {
  if (!L) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  cudaStream_t s = (cudaStream_t)stream;
  const int c = L->cur;
  MST_TRY(mst_ensure_csc(L, s));
  validate_rows<<<blocks_for(L->O, 128), 128, 0, s>>>(L->row_ptr[c], L->col_idx[c], L->bits[c], L->O, L->I, L->wpr,
                                                     L->nnz, L->flags); MST_COUNT_LAUNCH();
  validate_cols<<<blocks_for(L->I, 128), 128, 0, s>>>(L->col_ptr, L->row_idx, L->perm, L->row_ptr[c], L->col_idx[c],
                                                     L->O, L->I, L->nnz, L->flags); MST_COUNT_LAUNCH();
  MST_CUDA_TRY(cudaGetLastError());
  int32_t f = 0;
  MST_CUDA_TRY(cudaMemcpyAsync(&f, L->flags, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  MST_CUDA_TRY(cudaStreamSynchronize(s));
  if (f) MST_CUDA_TRY(cudaMemsetAsync(L->flags, 0, sizeof(int32_t), s));  // reported once, then cleared
  if (f & MST_FLAG_CORRUPT) return MST_ERR_CORRUPT;
  if (f & MST_FLAG_NONFINITE) return MST_ERR_NONFINITE;
  return MST_OK;
}

// ---- allocation-free mask -> CSR ------------------------------------------------------------------------------------
// Same popcount / scan / fill pipeline as mst_pack, but with no handle and no allocation: the mask words, their
// popcounts, the scan and the scan partials live in one file-scope device array that every GPU loading this library
// holds until the process exits.
namespace {

constexpr int64_t NOALLOC_MAX_NUMEL = (int64_t)1 << 22;  // 4 194 304 entries, e.g. a 4096 x 1024 layer
constexpr int64_t NOALLOC_MAX_WORDS = (int64_t)1 << 18;  // >= numel/32 + rows for every shape accepted below
constexpr int64_t NOALLOC_SUMS = NOALLOC_MAX_WORDS / SCAN_TILE + 2;
constexpr size_t NOALLOC_OFF_BITS = 0;
constexpr size_t NOALLOC_OFF_CNT = NOALLOC_OFF_BITS + 4 * (size_t)NOALLOC_MAX_WORDS;
constexpr size_t NOALLOC_OFF_SCAN = NOALLOC_OFF_CNT + 4 * (size_t)(NOALLOC_MAX_WORDS + 64);
constexpr size_t NOALLOC_OFF_SUMS = NOALLOC_OFF_SCAN + 4 * (size_t)(NOALLOC_MAX_WORDS + 64);
constexpr size_t NOALLOC_BYTES = NOALLOC_OFF_SUMS + 4 * (size_t)(NOALLOC_SUMS + 62);

static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_BYTES];

constexpr int NOALLOC_MAX_DEVICES = 64;
unsigned char* g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {};

// Device address of the scratch array on the current device.  g_noalloc_scratch itself is only a host-side handle
// for the symbol: the address a kernel can use has to be asked for, once per device, with that device current.
mst_status_t noalloc_scratch(unsigned char** out) {
  int devi = -1;
  MST_CUDA_TRY(cudaGetDevice(&devi));
  if (devi < 0 || devi >= NOALLOC_MAX_DEVICES) return MST_ERR_INVALID_ARG;
  if (!g_noalloc_ptr[devi]) {
    void* p = nullptr;
    MST_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    if (!p) return MST_ERR_CUDA;
    g_noalloc_ptr[devi] = (unsigned char*)p;
  }
  *out = g_noalloc_ptr[devi];
  return MST_OK;
}

// one warp per mask word, lane = bit; entries at positions >= cap are counted but not written
template <typename V>
__global__ void fill_csr_external(const uint32_t* __restrict__ bits, const int32_t* __restrict__ wscan, int O, int I,
                                  int wpr, const V* __restrict__ dense_W, int64_t ldw, int64_t cap,
                                  int32_t* __restrict__ row_ptr, int32_t* __restrict__ col_idx, V* __restrict__ vals) {
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const int64_t nwords = (int64_t)O * wpr;
  if (w >= nwords) return;
  const int o = (int)(w / wpr), wc = (int)(w % wpr);
  const uint32_t b = bits[w];
  const int32_t base = wscan[w];
  if (wc == 0 && lane == 0) {
    row_ptr[o] = base;
    if (o == O - 1) row_ptr[O] = wscan[nwords];
  }
  if ((b >> lane) & 1u) {
    const int64_t pos = (int64_t)base + __popc(b & lanemask_lt());
    if (pos < cap) {
      const int c = wc * 32 + lane;
      col_idx[pos] = c;
      vals[pos] = dense_W[(int64_t)o * ldw + c];
    }
  }
}

}  // namespace

extern "C" mst_status_t mst_mask_to_csr_noalloc(int32_t O, int32_t I, mst_dtype_t dtype, const void* W_dense,
                                                int64_t ldw, const uint8_t* mask, int64_t nnz_capacity,
                                                int32_t* row_ptr, int32_t* col_idx, void* vals, mst_stream_t stream) {
  if (!W_dense || !mask || !row_ptr || !col_idx || !vals || nnz_capacity < 0) return MST_ERR_INVALID_ARG;
  if (dtype != MST_F32 && dtype != MST_BF16) return MST_ERR_DTYPE;
  if (O < 1 || I < 1 || O > 65535 || I > 65535 || ldw < I) return MST_ERR_SHAPE;
  const int wpr = (I + 31) / 32;
  const int64_t nwords = (int64_t)O * wpr;
  if ((int64_t)O * I > NOALLOC_MAX_NUMEL || nwords > NOALLOC_MAX_WORDS) return MST_ERR_CAPACITY;
  unsigned char* base = nullptr;
  MST_TRY(noalloc_scratch(&base));
  uint32_t* bits = (uint32_t*)(base + NOALLOC_OFF_BITS);
  int32_t* cnt = (int32_t*)(base + NOALLOC_OFF_CNT);
  int32_t* scan = (int32_t*)(base + NOALLOC_OFF_SCAN);
  int32_t* sums = (int32_t*)(base + NOALLOC_OFF_SUMS);
  cudaStream_t s = (cudaStream_t)stream;
  // every word of the scratch that the later kernels read is written first by this call: nothing needs clearing
  mask_bytes_to_bits<<<blocks_for(nwords * 32, 256), 256, 0, s>>>(mask, O, I, wpr, bits); MST_COUNT_LAUNCH();
  popc_words<<<blocks_for(nwords, 256), 256, 0, s>>>(bits, nwords, cnt); MST_COUNT_LAUNCH();
  MST_TRY(mst_scan_i32(cnt, scan, nwords, sums, s));
  const unsigned grid = blocks_for(nwords * 32, 256);
  if (dtype == MST_F32)
    { fill_csr_external<float><<<grid, 256, 0, s>>>(bits, scan, O, I, wpr, (const float*)W_dense, ldw, nnz_capacity,
                                                  row_ptr, col_idx, (float*)vals); MST_COUNT_LAUNCH(); }
  else
    { fill_csr_external<uint16_t><<<grid, 256, 0, s>>>(bits, scan, O, I, wpr, (const uint16_t*)W_dense, ldw, nnz_capacity,
                                                     row_ptr, col_idx, (uint16_t*)vals); MST_COUNT_LAUNCH(); }
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}
