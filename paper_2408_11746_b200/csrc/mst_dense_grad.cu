// Dense gradient for gradient-based growth:  G[o, i] = sum_t dY[t, o] * X[t, i]   (fp32 out).
//
// bf16 operands with 16-byte-aligned rows go to the tensor cores (mst_tc_gemm.cu): both operands are MN-major there
// (dY is [T x O], X is [T x I], the contraction runs over T), the token range is split across blocks when the output
// has too few tiles to fill the GPU, and the partial sums are added in a fixed order.
// Everything else (fp32, odd leading dimensions) uses the CUDA-core tiled contraction below (fp32 accumulate): 64 x 64
// output tile per block, 16-token slices staged in shared memory in their natural layout, 4 x 4 outputs per thread.
#include "mst_internal.cuh"
#include "mst_tc_gemm.cuh"

namespace {

constexpr int TM = 64, TN = 64, TK = 16;

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const uint16_t* p) { return __uint_as_float(((uint32_t)*p) << 16); }

template <typename T>
__global__ void __launch_bounds__(256)
dense_grad_kernel(const T* __restrict__ dY, int64_t lddy, const T* __restrict__ X, int64_t ldx, int64_t T_total, int O,
                  int I, float* __restrict__ G) {
  __shared__ __align__(16) float As[TK][TM];
  __shared__ __align__(16) float Bs[TK][TN];
  const int o0 = blockIdx.y * TM, i0 = blockIdx.x * TN;
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  const int lk = threadIdx.x >> 4, lc = (threadIdx.x & 15) * 4;  // loader: slice row, first of 4 columns
  float acc[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;

  for (int64_t t0 = 0; t0 < T_total; t0 += TK) {
    const int64_t t = t0 + lk;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int o = o0 + lc + j, i = i0 + lc + j;
      As[lk][lc + j] = (t < T_total && o < O) ? ldf(dY + t * lddy + o) : 0.f;
      Bs[lk][lc + j] = (t < T_total && i < I) ? ldf(X + t * ldx + i) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(av[r], bv[c], acc[r][c]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int o = o0 + ty * 4 + r;
    if (o >= O) continue;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int i = i0 + tx * 4 + c;
      if (i < I) G[(int64_t)o * I + i] = acc[r][c];
    }
  }
}

}  // namespace

extern "C" mst_status_t mst_dense_grad(const void* dY, int64_t lddy, const void* X, int64_t ldx, int64_t T,
                                       int32_t out_features, int32_t in_features, mst_dtype_t dtype, float* G,
                                       mst_stream_t stream) {
  if (!G || T < 0 || out_features <= 0 || in_features <= 0 || (T > 0 && (!dY || !X))) return MST_ERR_INVALID_ARG;
  if (dtype != MST_F32 && dtype != MST_BF16) return MST_ERR_DTYPE;
  if (lddy < out_features || ldx < in_features) return MST_ERR_SHAPE;
  cudaStream_t s = (cudaStream_t)stream;
  if (T == 0) {
    MST_CUDA_TRY(cudaMemsetAsync(G, 0, sizeof(float) * (size_t)out_features * in_features, s));
    return MST_OK;
  }
  if (dtype == MST_BF16 && mst_tc_gemm_usable(dY, lddy, X, ldx) && ((reinterpret_cast<uintptr_t>(G) & 15u) == 0)) {
    mst_tc_gemm_args a = {};
    a.A = dY; a.lda = lddy; a.a_mn_major = 1;
    a.B = X; a.ldb = ldx; a.b_mn_major = 1;
    a.M = out_features; a.N = in_features; a.K = T;
    a.epilogue = MST_TC_OUT_F32;
    a.out = G; a.ldc = in_features;
    a.splits = 0;
    return mst_tc_gemm(a, s);
  }
  dim3 grid((unsigned)((in_features + TN - 1) / TN), (unsigned)((out_features + TM - 1) / TM));
  if (dtype == MST_F32)
    { dense_grad_kernel<float><<<grid, 256, 0, s>>>((const float*)dY, lddy, (const float*)X, ldx, T, out_features,
                                                 in_features, G); MST_COUNT_LAUNCH(); }
  else
    { dense_grad_kernel<uint16_t><<<grid, 256, 0, s>>>((const uint16_t*)dY, lddy, (const uint16_t*)X, ldx, T,
                                                    out_features, in_features, G); MST_COUNT_LAUNCH(); }
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}
