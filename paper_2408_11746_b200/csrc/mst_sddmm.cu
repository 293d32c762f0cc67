// Sampled dense-dense product on the mask:  dW[k] = sum_t dY[t, o_k] * X[t, i_k]  for every stored entry k.
//
// A block owns a ROWS x COLS window of the weight matrix and walks over all tokens in tiles of TOK.  For each token
// tile both operand tiles are staged feature-major in shared memory (Ds[row][token], Xs[col][token]) so that a lane
// owning 8 consecutive tokens fetches its operands with 128-bit shared loads.  The window's stored entries are
// listed once (row-local, column-local) in shared memory; a warp takes them 32 at a time: every lane forms its
// 8-token partial dot product of each of the 32 entries, then a 31-shuffle transposing reduction leaves the full
// sum of entry j in lane j, which adds it to that entry's fp32 accumulator in shared memory.  The upstream-gradient
// operands of a row stay in registers while consecutive entries share the row.  Every entry is owned by exactly one
// warp and one lane, the token order is fixed: no atomics, deterministic.
#include "mst_bits.cuh"
#include "mst_internal.cuh"
#include "mst_tc_gemm.cuh"

namespace {

constexpr int TOK = 256;
constexpr int ROWS = 64;
constexpr int COLS = 64;
constexpr int WARPS = 8;
constexpr int RPW = ROWS / WARPS;
constexpr int LIST_CAP = ROWS * COLS;

__device__ __forceinline__ void load8(float (&v)[8], const float* p) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(float (&v)[8], const uint16_t* p) {
  const uint4 q = *reinterpret_cast<const uint4*>(p);
  v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xFFFF0000u);
  v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xFFFF0000u);
  v[4] = __uint_as_float(q.z << 16); v[5] = __uint_as_float(q.z & 0xFFFF0000u);
  v[6] = __uint_as_float(q.w << 16); v[7] = __uint_as_float(q.w & 0xFFFF0000u);
}

// Stage `ncols` (<= 64) feature columns starting at c0 of tokens [t0, t0+TOK) into S[c][token]; zero fill outside.
template <typename T>
__device__ __forceinline__ void stage64(T* __restrict__ S, const T* __restrict__ in, int64_t ld, int64_t T_total, int C,
                                        int64_t t0, int c0, bool vec_ok) {
  constexpr int VEC = 16 / (int)sizeof(T);
  const int tt = threadIdx.x;
  const int64_t t = t0 + tt;
  const bool row_ok = t < T_total;
  const T* src = in + t * ld + c0;
  if (vec_ok) {
#pragma unroll 4
    for (int v = 0; v < COLS / VEC; ++v) {
      uint4 q = make_uint4(0, 0, 0, 0);
      if (row_ok && c0 + v * VEC < C) q = *reinterpret_cast<const uint4*>(src + v * VEC);
      const T* e = reinterpret_cast<const T*>(&q);
#pragma unroll
      for (int j = 0; j < VEC; ++j) S[(v * VEC + j) * TOK + tt] = e[j];
    }
  } else {
    for (int c = 0; c < COLS; ++c) {
      T x = T(0);
      if (row_ok && c0 + c < C) x = src[c];
      S[c * TOK + tt] = x;
    }
  }
}

__device__ __forceinline__ int lower_bound_u16(const uint16_t* __restrict__ a, int lo, int hi, int key) {
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if ((int)a[mid] < key) lo = mid + 1; else hi = mid;
  }
  return lo;
}

template <typename T>
__global__ void __launch_bounds__(WARPS * 32)
sddmm_window_kernel(const int32_t* __restrict__ row_ptr, const uint16_t* __restrict__ col_idx,
                    const T* __restrict__ dY, int64_t lddy, const T* __restrict__ X, int64_t ldx, int64_t T_total, int O,
                    int I, float* __restrict__ dW, int vec_x, int vec_dy) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  T* Xs = reinterpret_cast<T*>(smem_raw);                       // [COLS][TOK]
  T* Ds = Xs + COLS * TOK;                                      // [ROWS][TOK]
  float* accS = reinterpret_cast<float*>(Ds + ROWS * TOK);      // [LIST_CAP]
  uint16_t* list = reinterpret_cast<uint16_t*>(accS + LIST_CAP);  // [LIST_CAP]  (row_local << 8) | col_local
  __shared__ int ks[ROWS];          // CSR position of the row's first entry inside the window
  __shared__ int lstart[ROWS + 1];  // list offset of each row

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int o0 = blockIdx.x * ROWS, c0 = blockIdx.y * COLS;

  // ---- list the stored entries of the window
  if (threadIdx.x < ROWS) {
    const int o = o0 + threadIdx.x;
    int a = 0, b = 0;
    if (o < O) {
      const int lo = row_ptr[o], hi = row_ptr[o + 1];
      a = lower_bound_u16(col_idx, lo, hi, c0);
      b = lower_bound_u16(col_idx, a, hi, c0 + COLS);
    }
    ks[threadIdx.x] = a;
    lstart[threadIdx.x + 1] = b - a;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    lstart[0] = 0;
    for (int r = 0; r < ROWS; ++r) {
      const int c = lstart[r + 1];
      lstart[r + 1] = run + c;
      run += c;
    }
  }
  __syncthreads();
  const int L = lstart[ROWS];
  if (L == 0) return;
  for (int rr = 0; rr < RPW; ++rr) {
    const int rl = warp * RPW + rr;
    const int a = ks[rl], n = lstart[rl + 1] - lstart[rl], base = lstart[rl];
    for (int e = lane; e < n; e += 32) list[base + e] = (uint16_t)((rl << 8) | ((int)col_idx[a + e] - c0));
  }
  for (int e = threadIdx.x; e < L; e += WARPS * 32) accS[e] = 0.f;

  const int groups = (L + 31) >> 5;
  for (int64_t t0 = 0; t0 < T_total; t0 += TOK) {
    __syncthreads();
    stage64<T>(Xs, X, ldx, T_total, I, t0, c0, vec_x != 0);
    stage64<T>(Ds, dY, lddy, T_total, O, t0, o0, vec_dy != 0);
    __syncthreads();
    for (int g = warp; g < groups; g += WARPS) {
      float p[32];
      float dy[8];
      int cur_row = -1;
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        p[j] = 0.f;
        const int e = g * 32 + j;
        if (e < L) {
          const int ent = list[e];
          const int rl = ent >> 8, cl = ent & 0xFF;
          if (rl != cur_row) {
            load8(dy, Ds + rl * TOK + lane * 8);
            cur_row = rl;
          }
          float x[8];
          load8(x, Xs + (cl & (COLS - 1)) * TOK + lane * 8);
          float s = dy[0] * x[0];
#pragma unroll
          for (int i = 1; i < 8; ++i) s = fmaf(dy[i], x[i], s);
          p[j] = s;
        }
      }
      // transposing reduction: afterwards p[0] in lane j is the sum over all lanes of entry j
#pragma unroll
      for (int h = 16; h >= 1; h >>= 1) {
        const bool up = (lane & h) != 0;
#pragma unroll
        for (int i = 0; i < h; ++i) {
          const float send = up ? p[i] : p[i + h];
          const float keep = up ? p[i + h] : p[i];
          p[i] = keep + __shfl_xor_sync(0xffffffffu, send, h);
        }
      }
      const int e = g * 32 + lane;
      if (e < L) accS[e] += p[0];
    }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < L; e += WARPS * 32) {
    const int rl = list[e] >> 8;
    dW[ks[rl] + (e - lstart[rl])] = accS[e];
  }
}

// dW on the mask read out of a dense gradient: one warp per mask word, lane = column.
__global__ void sample_dense_kernel(const uint32_t* __restrict__ bits, const int32_t* __restrict__ wscan, int O, int I,
                                    int wpr, const float* __restrict__ G, float* __restrict__ dW) {
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= (int64_t)O * wpr) return;
  const uint32_t b = bits[w];
  if (!((b >> lane) & 1u)) return;
  const unsigned wu = (unsigned)w;
  const int o = (int)(wu / (unsigned)wpr), c = (int)(wu - (unsigned)o * (unsigned)wpr) * 32 + lane;
  dW[wscan[w] + __popc(b & mst_lanemask_lt())] = G[(int64_t)o * I + c];
}

template <typename T>
mst_status_t launch(const mst_layer* L, const void* dY, int64_t lddy, const void* X, int64_t ldx, int64_t T_total,
                    float* dW, cudaStream_t s) {
  constexpr int VEC = 16 / (int)sizeof(T);
  const size_t smem = (size_t)(COLS + ROWS) * TOK * sizeof(T) + (size_t)LIST_CAP * (4 + 2);
  MST_CUDA_TRY(cudaFuncSetAttribute(sddmm_window_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const int vec_x = (ldx % VEC == 0) && (L->I % VEC == 0) && ((reinterpret_cast<uintptr_t>(X) & 15u) == 0);
  const int vec_dy = (lddy % VEC == 0) && (L->O % VEC == 0) && ((reinterpret_cast<uintptr_t>(dY) & 15u) == 0);
  dim3 grid((unsigned)((L->O + ROWS - 1) / ROWS), (unsigned)((L->I + COLS - 1) / COLS));
  const int c = L->cur;
  sddmm_window_kernel<T><<<grid, WARPS * 32, smem, s>>>(L->row_ptr[c], L->col_idx[c], (const T*)dY, lddy, (const T*)X,
                                                      ldx, T_total, L->O, L->I, dW, vec_x, vec_dy);
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

}  // namespace

mst_status_t mst_launch_sddmm(const mst_layer* L, const void* dY, int64_t lddy, const void* X, int64_t ldx, int64_t T,
                              float* dW, cudaStream_t s) {
  if (L->nnz == 0) return MST_OK;
  if (T == 0) {
    MST_CUDA_TRY(cudaMemsetAsync(dW, 0, sizeof(float) * L->nnz, s));
    return MST_OK;
  }
  // Tensor-core path: the dense contraction dY^T X with an epilogue that keeps only the entries under the mask and
  // writes them to their CSR positions; the token range is split when the output has few tiles.
  if (mst_use_tensor_path(L) && mst_tc_gemm_usable(dY, lddy, X, ldx)) {
    const int c = L->cur;
    mst_tc_gemm_args a = {};
    a.A = dY; a.lda = lddy; a.a_mn_major = 1;
    a.B = X; a.ldb = ldx; a.b_mn_major = 1;
    a.M = L->O; a.N = L->I; a.K = T;
    a.epilogue = MST_TC_OUT_SAMPLED;
    a.out = dW;
    a.bits = L->bits[c]; a.wscan = L->wscan[c]; a.wpr = L->wpr; a.nnz = L->nnz;
    a.splits = 0;
    return mst_tc_gemm(a, s);
  }
  if (L->dtype == MST_F32) return launch<float>(L, dY, lddy, X, ldx, T, dW, s);
  return launch<uint16_t>(L, dY, lddy, X, ldx, T, dW, s);
}

extern "C" mst_status_t mst_sddmm_dw(const mst_layer_t* L, const void* dY, int64_t lddy, const void* X, int64_t ldx,
                                     int64_t T, float* dW_vals, mst_stream_t stream) {
  if (!L || T < 0 || !dW_vals || (T > 0 && (!dY || !X))) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  if (lddy < L->O || ldx < L->I) return MST_ERR_SHAPE;
  return mst_launch_sddmm(L, dY, lddy, X, ldx, T, dW_vals, (cudaStream_t)stream);
}

extern "C" mst_status_t mst_sddmm_from_dense(const mst_layer_t* L, const float* G_dense, float* dW_vals,
                                             mst_stream_t stream) {
  if (!L || !G_dense || !dW_vals) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  if (L->nnz == 0) return MST_OK;
  const int c = L->cur;
  const int64_t threads = L->nwords * 32;
  sample_dense_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
      L->bits[c], L->wscan[c], L->O, L->I, L->wpr, G_dense, dW_vals);
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

extern "C" mst_status_t mst_dense_grad_dw(const mst_layer_t* L, const void* dY, int64_t lddy, const void* X, int64_t ldx,
                                          int64_t T, float* G_dense, float* dW_vals, mst_stream_t stream) {
  if (!L || !G_dense || !dW_vals) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  MST_TRY(mst_dense_grad(dY, lddy, X, ldx, T, L->O, L->I, L->dtype, G_dense, stream));
  return mst_sddmm_from_dense(L, G_dense, dW_vals, stream);
}
