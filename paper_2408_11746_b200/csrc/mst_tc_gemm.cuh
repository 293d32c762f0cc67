// Interface of the tcgen05 (5th-generation tensor core) bf16 contraction used for the dense gradient,
// the dense-tile SpMM path and the sampled weight gradient.  Internal to libmst.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "mst.h"

// C[M x N] = A * B^T-like contraction over K with fp32 accumulation in tensor memory.
//   A operand: K-major   -> A is stored [M x K] row-major (lda elements between rows), or
//              MN-major  -> A is stored [K x M] row-major (lda elements between K rows)
//   B operand: K-major   -> B is stored [N x K] row-major, or MN-major -> [K x N] row-major
// Epilogues:
//   MST_TC_OUT_BF16     C bf16 row-major [M x ldc]
//   MST_TC_OUT_F32      C fp32 row-major [M x ldc]; with splits > 1 writes partial sums to
//                       partial[split][M x N] (contiguous) which mst_tc_reduce then sums in a fixed order
//   MST_TC_OUT_SAMPLED  only entries under a bit mask are written, to their CSR position:
//                       out[wscan[w] + rank] for mask word w = m*wpr + n/32 (needs N-tile offsets multiple of 32)
enum { MST_TC_OUT_BF16 = 0, MST_TC_OUT_F32 = 1, MST_TC_OUT_SAMPLED = 2 };

// Element-wise step fused into the bf16 epilogue (GPT-2 MLP: fc1 -> GELU -> fc2, erf form):
//   GELU       out = gelu(acc), optionally pre = acc
//   GELU_GRAD  out = acc * gelu'(pre)
enum { MST_ACT_NONE = 0, MST_ACT_GELU = 1, MST_ACT_GELU_GRAD = 2 };

__host__ __device__ inline float mst_gelu(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752f)); }
__host__ __device__ inline float mst_gelu_grad(float x) {
  return 0.5f * (1.0f + erff(x * 0.70710678118654752f)) + x * 0.39894228040143268f * expf(-0.5f * x * x);
}

struct mst_tc_gemm_args {
  const void* A;
  int64_t lda;
  int a_mn_major;
  const void* B;
  int64_t ldb;
  int b_mn_major;
  int64_t M, N, K;
  int epilogue;
  void* out;
  int64_t ldc;
  int splits;            // 0 = choose; otherwise K is cut into this many contiguous ranges (F32 / SAMPLED epilogues);
                         // partial sums live in the process-wide scratch buffer and are added in a fixed order
  const uint32_t* bits;  // SAMPLED: mask words, wpr per row
  const int32_t* wscan;  // SAMPLED: exclusive popcount scan of the words
  int wpr;
  int64_t nnz;           // SAMPLED: number of stored entries (partial stride)
  int act;               // BF16 epilogue only: MST_ACT_NONE / MST_ACT_GELU / MST_ACT_GELU_GRAD
  void* pre;             // GELU: optional bf16 output for the pre-activation (may be NULL);
                         // GELU_GRAD: bf16 input holding the pre-activation the derivative is taken at
  int64_t ldpre;
};

// Returns MST_ERR_SHAPE when the operands cannot be described to the TMA unit (leading dimension or base address
// not 16-byte aligned); the caller then falls back to the CUDA-core kernel.
mst_status_t mst_tc_gemm(const mst_tc_gemm_args& a, cudaStream_t s);
bool mst_tc_gemm_usable(const void* A, int64_t lda, const void* B, int64_t ldb);

int mst_tc_pick_splits(int64_t works1, int64_t slots, int64_t kblocks, double out_bytes);

// Process-wide scratch buffer for handle-less entry points (grows on demand; growing synchronises the device).
// Calls that use it must not overlap on the GPU.
mst_status_t mst_workspace(size_t bytes, void** ptr);
// The same per purpose: split partial sums, feature-major activation columns of the structured-sparse path.
enum { MST_WS_SPLIT = 0, MST_WS_COLUMNS = 1, MST_WS_ATTENTION = 2, MST_WS_IMAGE = 3, MST_WS_KINDS = 4 };
mst_status_t mst_workspace_kind(int kind, size_t bytes, void** ptr);
