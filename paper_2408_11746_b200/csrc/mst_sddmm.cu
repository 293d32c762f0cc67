// Sampled dense-dense product on the mask:  dW[k] = sum_t dY[t, o_k] * X[t, i_k]  for every stored entry k.
//
// Both operands are first copied feature-major once per call (dYT[o][t], XT[i][t]).  A block owns a ROWS x COLS
// window of the weight matrix and walks over all tokens in tiles of TOK: for each token tile the two operand tiles
// (Ds[row][token], Xs[col][token]) arrive in shared memory through the TMA unit (cp.async.bulk.tensor, this GPU's
// memory only, no multicast), so that a lane owning 8 consecutive tokens fetches its operands with 128-bit shared
// loads.  The window's stored entries are listed once (row-local, column-local) in shared memory; a warp takes them
// 32 at a time: every lane forms its 8-token partial dot product of each of the 32 entries (bf16 layers: with the
// mixed-precision FMA, bf16 x bf16 + fp32, no unpacking), then a 31-shuffle transposing reduction leaves the full
// sum of entry j in lane j, which adds it to that entry's fp32 accumulator in shared memory.  The upstream-gradient
// operands of a row stay in registers while consecutive entries share the row.  Every entry is owned by exactly one
// warp and one lane, the token order is fixed: no atomics, deterministic.
#include <cuda.h>

#include "mst_bits.cuh"
#include "mst_internal.cuh"
#include "mst_tc_gemm.cuh"
#include "mst_tc_ptx.cuh"

// feature-major copies and their TMA description (mst_spmm.cu)
mst_status_t mst_feature_major_copy(const void* in, int64_t ldin, int64_t T, int C, mst_dtype_t dtype, void* out, int64_t ldt,
                                    cudaStream_t s);
bool mst_feature_major_map(CUtensorMap* tm, const void* base, int64_t T, int C, int64_t ldt, mst_dtype_t dtype, int box_tokens,
                           int box_features);

namespace {

constexpr int TOK = 256;
constexpr int ROWS = 64;
constexpr int COLS = 64;
constexpr int WARPS = 8;
constexpr int RPW = ROWS / WARPS;
constexpr int LIST_CAP = ROWS * COLS;

__device__ int g_sddmm_error = 0;  // sticky: a bounded wait expired

// 8 consecutive tokens of one feature, as stored
template <typename T>
struct Vec8;
template <>
struct Vec8<float> {
  float4 a, b;
  __device__ __forceinline__ void load(const float* p) {
    a = *reinterpret_cast<const float4*>(p);
    b = *reinterpret_cast<const float4*>(p + 4);
  }
};
template <>
struct Vec8<uint16_t> {
  uint4 q;
  __device__ __forceinline__ void load(const uint16_t* p) { q = *reinterpret_cast<const uint4*>(p); }
};
__device__ __forceinline__ float dot8(const Vec8<float>& d, const Vec8<float>& x) {
  float s0 = d.a.x * x.a.x, s1 = d.a.y * x.a.y;
  s0 = fmaf(d.a.z, x.a.z, s0); s1 = fmaf(d.a.w, x.a.w, s1);
  s0 = fmaf(d.b.x, x.b.x, s0); s1 = fmaf(d.b.y, x.b.y, s1);
  s0 = fmaf(d.b.z, x.b.z, s0); s1 = fmaf(d.b.w, x.b.w, s1);
  return s0 + s1;
}
// exact bf16 products accumulated in fp32 (mixed-precision FMA of sm_100), two chains of four
__device__ __forceinline__ float dot8(const Vec8<uint16_t>& d, const Vec8<uint16_t>& x) {
  const uint32_t dw[4] = {d.q.x, d.q.y, d.q.z, d.q.w}, xw[4] = {x.q.x, x.q.y, x.q.z, x.q.w};
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint16_t dl, dh, xl, xh;
    asm("mov.b32 {%0, %1}, %2;" : "=h"(dl), "=h"(dh) : "r"(dw[j]));
    asm("mov.b32 {%0, %1}, %2;" : "=h"(xl), "=h"(xh) : "r"(xw[j]));
    asm("fma.rn.f32.bf16 %0, %1, %2, %0;" : "+f"(s0) : "h"(dl), "h"(xl));
    asm("fma.rn.f32.bf16 %0, %1, %2, %0;" : "+f"(s1) : "h"(dh), "h"(xh));
  }
  return s0 + s1;
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
sddmm_window_kernel(const __grid_constant__ CUtensorMap tmDY, const __grid_constant__ CUtensorMap tmX,
                    const int32_t* __restrict__ row_ptr, const uint16_t* __restrict__ col_idx, int64_t T_total, int O,
                    int I, float* __restrict__ dW) {
  using namespace mst_ptx;
  constexpr uint32_t TILE_BYTES = (uint32_t)(COLS * TOK * sizeof(T));
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 127u) & ~127u;
  unsigned char* tiles = smem_raw + (tiles_base - raw);
  T* Xs = reinterpret_cast<T*>(tiles);                             // [COLS][TOK]
  T* Ds = reinterpret_cast<T*>(tiles + TILE_BYTES);                // [ROWS][TOK]
  float* accS = reinterpret_cast<float*>(tiles + 2 * TILE_BYTES);  // [LIST_CAP]
  uint16_t* list = reinterpret_cast<uint16_t*>(accS + LIST_CAP);   // [LIST_CAP]  (row_local << 8) | col_local
  __shared__ int ks[ROWS];          // CSR position of the row's first entry inside the window
  __shared__ int lstart[ROWS + 1];  // list offset of each row
  __shared__ uint64_t bar;
  __shared__ int abort_sh;
  volatile int* abort_flag = &abort_sh;

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int o0 = blockIdx.x * ROWS, c0 = blockIdx.y * COLS;
  if (threadIdx.x == 0) {
    abort_sh = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }

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
  uint32_t ph = 0;
  for (int64_t t0 = 0; t0 < T_total; t0 += TOK) {
    __syncthreads();  // the previous tiles have been read by every warp; list and accumulators are initialised
    if (threadIdx.x == 0) {
      mbar_expect_tx(smem_u32(&bar), 2 * TILE_BYTES);
      tma_load_2d(tiles_base, &tmX, (int)t0, c0, smem_u32(&bar));
      tma_load_2d(tiles_base + TILE_BYTES, &tmDY, (int)t0, o0, smem_u32(&bar));
    }
    if (!mst_ptx::mbar_wait(smem_u32(&bar), ph, abort_flag, &g_sddmm_error)) break;
    ph ^= 1u;
    for (int g = warp; g < groups; g += WARPS) {
      float p[32];
      Vec8<T> dy;
      int cur_row = -1;
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        p[j] = 0.f;
        const int e = g * 32 + j;
        if (e < L) {
          const int ent = list[e];
          const int rl = ent >> 8, cl = ent & 0xFF;
          if (rl != cur_row) {
            dy.load(Ds + rl * TOK + lane * 8);
            cur_row = rl;
          }
          Vec8<T> x;
          x.load(Xs + (cl & (COLS - 1)) * TOK + lane * 8);
          p[j] = dot8(dy, x);
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
  // feature-major copies of both operands in the per-device column scratch: [I x ldt] then [O x ldt]
  const int64_t ldt = (T_total + 63) / 64 * 64;
  void* ws = nullptr;
  MST_TRY(mst_workspace_kind(MST_WS_COLUMNS, (size_t)(L->I + L->O) * ldt * sizeof(T), &ws));
  T* XT = (T*)ws;
  T* dYT = XT + (size_t)L->I * ldt;
  MST_TRY(mst_feature_major_copy(X, ldx, T_total, L->I, L->dtype, XT, ldt, s));
  MST_TRY(mst_feature_major_copy(dY, lddy, T_total, L->O, L->dtype, dYT, ldt, s));
  CUtensorMap tmX, tmDY;
  if (!mst_feature_major_map(&tmX, XT, T_total, L->I, ldt, L->dtype, TOK, COLS) ||
      !mst_feature_major_map(&tmDY, dYT, T_total, L->O, ldt, L->dtype, TOK, ROWS))
    return MST_ERR_SHAPE;
  const size_t smem = (size_t)(COLS + ROWS) * TOK * sizeof(T) + (size_t)LIST_CAP * (4 + 2) + 128;
  MST_CUDA_TRY(cudaFuncSetAttribute(sddmm_window_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid((unsigned)((L->O + ROWS - 1) / ROWS), (unsigned)((L->I + COLS - 1) / COLS));
  const int c = L->cur;
  sddmm_window_kernel<T><<<grid, WARPS * 32, smem, s>>>(tmDY, tmX, L->row_ptr[c], L->col_idx[c], T_total, L->O, L->I, dW); MST_COUNT_LAUNCH();
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

}  // namespace

mst_status_t mst_sddmm_error_flags(int32_t* flags) {
  int v = 0;
  MST_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_sddmm_error, sizeof(int)));
  *flags = v;
  return MST_OK;
}

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
      L->bits[c], L->wscan[c], L->O, L->I, L->wpr, G_dense, dW_vals); MST_COUNT_LAUNCH();
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
