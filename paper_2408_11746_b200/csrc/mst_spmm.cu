// Row-panel SpMM on the CUDA cores:  out[t, r] = sum_{k in row r} val(k) * in[t, idx[k]].
//
// Forward uses the CSR arrays (r = output feature, idx = input feature); the input gradient uses the CSC view
// (r = input feature, idx = output feature, values fetched through the CSC->CSR permutation), so both are gathers
// with a fixed summation order: no floating-point atomics, run-to-run identical results.
//
// A block owns TOK tokens x PANEL rows.  The activation tile is staged feature-major in shared memory, one column
// chunk at a time (Xs[c][token]), so that a lane that owns 8 consecutive tokens fetches its 8 operands of one
// nonzero with a single 128-bit (bf16) or two 128-bit (fp32) shared loads.  A warp owns PANEL/8 rows and walks each
// row's nonzeros with a cursor that advances chunk by chunk (columns ascend inside a row); indices and values are
// loaded 32 at a time, coalesced, and broadcast with shuffles.  Accumulation is fp32 in registers; the output tile
// goes through shared memory so that global stores are contiguous along the feature dimension.
#include "mst_internal.cuh"
#include "mst_tc_gemm.cuh"

namespace {

constexpr int TOK = 256;    // tokens per block (8 per lane)
constexpr int PANEL = 64;   // rows per block
constexpr int WARPS = 8;
constexpr int RPW = PANEL / WARPS;
constexpr int OS_LD = PANEL + 1;

template <typename T>
struct Cfg;
template <>
struct Cfg<float> {
  static constexpr int KC = 64;
  static constexpr int VEC = 4;
};
template <>
struct Cfg<uint16_t> {
  static constexpr int KC = 128;
  static constexpr int VEC = 8;
};

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(uint16_t v) { return __uint_as_float(((uint32_t)v) << 16); }

__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
// fp32 -> bf16, round to nearest even (finite inputs)
__device__ __forceinline__ void store_out(uint16_t* p, float v) {
  uint32_t u = __float_as_uint(v);
  if ((u & 0x7F800000u) != 0x7F800000u) u += 0x7FFFu + ((u >> 16) & 1u);
  *p = (uint16_t)(u >> 16);
}

__device__ __forceinline__ void fma8(float (&acc)[8], float w, const float* xs) {
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
__device__ __forceinline__ void fma8(float (&acc)[8], float w, const uint16_t* xs) {
  const uint4 v = *reinterpret_cast<const uint4*>(xs);
  acc[0] = fmaf(w, __uint_as_float(v.x << 16), acc[0]);
  acc[1] = fmaf(w, __uint_as_float(v.x & 0xFFFF0000u), acc[1]);
  acc[2] = fmaf(w, __uint_as_float(v.y << 16), acc[2]);
  acc[3] = fmaf(w, __uint_as_float(v.y & 0xFFFF0000u), acc[3]);
  acc[4] = fmaf(w, __uint_as_float(v.z << 16), acc[4]);
  acc[5] = fmaf(w, __uint_as_float(v.z & 0xFFFF0000u), acc[5]);
  acc[6] = fmaf(w, __uint_as_float(v.w << 16), acc[6]);
  acc[7] = fmaf(w, __uint_as_float(v.w & 0xFFFF0000u), acc[7]);
}

// Stage columns [c0, c0+KC) of tokens [t0, t0+TOK) into Xs[c][token]; out-of-range elements become 0.
template <typename T>
__device__ __forceinline__ void stage_tile(T* __restrict__ Xs, const T* __restrict__ in, int64_t ld, int64_t T_total,
                                           int C, int64_t t0, int c0, bool vec_ok) {
  constexpr int KC = Cfg<T>::KC, VEC = Cfg<T>::VEC;
  const int tt = threadIdx.x;
  const int64_t t = t0 + tt;
  const bool row_ok = t < T_total;
  const T* src = in + t * ld + c0;
  if (vec_ok) {
#pragma unroll 4
    for (int v = 0; v < KC / VEC; ++v) {
      uint4 q = make_uint4(0, 0, 0, 0);
      if (row_ok && c0 + v * VEC < C) q = *reinterpret_cast<const uint4*>(src + v * VEC);
      const T* e = reinterpret_cast<const T*>(&q);
#pragma unroll
      for (int j = 0; j < VEC; ++j) Xs[(v * VEC + j) * TOK + tt] = e[j];
    }
  } else {
    for (int c = 0; c < KC; ++c) {
      T x = T(0);
      if (row_ok && c0 + c < C) x = src[c];
      Xs[c * TOK + tt] = x;
    }
  }
}

template <typename T, bool PERM>
__global__ void __launch_bounds__(WARPS * 32, 2)
spmm_panel_kernel(const int32_t* __restrict__ ptr, const uint16_t* __restrict__ idx, const T* __restrict__ vals,
                  const int32_t* __restrict__ perm, const T* __restrict__ in, int64_t ldin, T* __restrict__ out,
                  int64_t ldout, int64_t T_total, int R_total, int C, int vec_ok) {
  constexpr int KC = Cfg<T>::KC;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  T* Xs = reinterpret_cast<T*>(smem_raw);
  float* Os = reinterpret_cast<float*>(smem_raw);

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int r_base = blockIdx.x * PANEL + warp * RPW;
  const int64_t t0 = (int64_t)blockIdx.y * TOK;

  int32_t kcur[RPW], kend[RPW];
  float acc[RPW][8];
#pragma unroll
  for (int rr = 0; rr < RPW; ++rr) {
    const int r = r_base + rr;
    kcur[rr] = r < R_total ? ptr[r] : 0;
    kend[rr] = r < R_total ? ptr[r + 1] : 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[rr][j] = 0.f;
  }

  for (int c0 = 0; c0 < C; c0 += KC) {
    __syncthreads();  // previous chunk fully consumed
    stage_tile<T>(Xs, in, ldin, T_total, C, t0, c0, vec_ok != 0);
    __syncthreads();
    const uint32_t c_end = (uint32_t)(c0 + KC);
#pragma unroll
    for (int rr = 0; rr < RPW; ++rr) {
      int32_t k = kcur[rr];
      const int32_t e = kend[rr];
      while (k < e) {
        const int32_t kk = k + lane;
        const uint32_t ci = kk < e ? (uint32_t)idx[kk] : 0xFFFFFFFFu;
        const bool inb = ci < c_end;
        const unsigned m = __ballot_sync(0xffffffffu, inb);
        const int n = __popc(m);  // columns ascend, so the in-chunk entries are the first n
        if (n == 0) break;
        float w = 0.f;
        if (inb) w = to_float(PERM ? vals[perm[kk]] : vals[kk]);
        const int cl = (int)ci - c0;
        for (int j = 0; j < n; ++j) {
          const int cj = __shfl_sync(0xffffffffu, cl, j);
          const float wj = __shfl_sync(0xffffffffu, w, j);
          fma8(acc[rr], wj, Xs + cj * TOK + lane * 8);
        }
        k += n;
        if (n < 32) break;
      }
      kcur[rr] = k;
    }
  }

  // epilogue: registers -> shared (token-permuted rows, conflict-free) -> global, contiguous along the rows
  __syncthreads();
#pragma unroll
  for (int rr = 0; rr < RPW; ++rr)
#pragma unroll
    for (int j = 0; j < 8; ++j) Os[(j * 32 + lane) * OS_LD + warp * RPW + rr] = acc[rr][j];
  __syncthreads();
  for (int i = threadIdx.x; i < TOK * PANEL; i += WARPS * 32) {
    const int tt = i / PANEL, rl = i % PANEL;
    const int64_t t = t0 + tt;
    const int r = blockIdx.x * PANEL + rl;
    if (t < T_total && r < R_total) store_out(out + t * ldout + r, Os[((tt & 7) * 32 + (tt >> 3)) * OS_LD + rl]);
  }
}

template <typename T>
constexpr size_t spmm_smem() {
  return (size_t)Cfg<T>::KC * TOK * sizeof(T) > (size_t)TOK * OS_LD * 4 ? (size_t)Cfg<T>::KC * TOK * sizeof(T)
                                                                      : (size_t)TOK * OS_LD * 4;
}

template <typename T, bool PERM>
mst_status_t launch(const int32_t* ptr, const uint16_t* idx, const void* vals, const int32_t* perm, const void* in,
                    int64_t ldin, void* out, int64_t ldout, int64_t T_total, int R_total, int C, cudaStream_t s) {
  const size_t smem = spmm_smem<T>();
  // per call: the attribute belongs to the current device's copy of the kernel
  MST_CUDA_TRY(cudaFuncSetAttribute(spmm_panel_kernel<T, PERM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  constexpr int VEC = Cfg<T>::VEC;
  const int vec_ok = (ldin % VEC == 0) && (C % VEC == 0) && ((reinterpret_cast<uintptr_t>(in) & 15u) == 0);
  dim3 grid((unsigned)((R_total + PANEL - 1) / PANEL), (unsigned)((T_total + TOK - 1) / TOK));
  spmm_panel_kernel<T, PERM><<<grid, WARPS * 32, smem, s>>>(ptr, idx, (const T*)vals, perm, (const T*)in, ldin, (T*)out,
                                                          ldout, T_total, R_total, C, vec_ok);
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
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
  act_rows_kernel<T><<<blocks, 256, 0, s>>>((T*)out, ldout, (const T*)pre, ldpre, rows, cols, act);
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

}  // namespace

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
    const uint16_t* image = L->dense_w;
    if (mst_tc_gemm_usable(in, ldin, image, L->I)) {
      MST_TRY(mst_densify(L, s));
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
    st = L->dtype == MST_F32
             ? launch<float, false>(L->row_ptr[c], L->col_idx[c], L->vals[c], nullptr, in, ldin, prod, ldprod, T, L->O, L->I, s)
             : launch<uint16_t, false>(L->row_ptr[c], L->col_idx[c], L->vals[c], nullptr, in, ldin, prod, ldprod, T, L->O, L->I, s);
  } else {
    MST_TRY(mst_ensure_csc(L, s));
    st = L->dtype == MST_F32
             ? launch<float, true>(L->col_ptr, L->row_idx, L->vals[c], L->perm, in, ldin, prod, ldprod, T, L->I, L->O, s)
             : launch<uint16_t, true>(L->col_ptr, L->row_idx, L->vals[c], L->perm, in, ldin, prod, ldprod, T, L->I, L->O, s);
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
