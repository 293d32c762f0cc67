// Handle management and the host-buffer convenience entry point of libmst.
#include "mst_internal.cuh"

#include <new>

std::atomic<long long> g_mst_launches{0};

namespace {

struct Carver {
  size_t off = 0;
  size_t take(size_t bytes) {
    const size_t at = off;
    off += (bytes + 255) & ~(size_t)255;
    return at;
  }
};

void free_staging(mst_layer* L) {
  cudaFree(L->stg_x);
  cudaFree(L->stg_dy);
  cudaFree(L->stg_y);
  cudaFree(L->stg_dx);
  cudaFree(L->stg_dw);
  L->stg_x = L->stg_dy = L->stg_y = L->stg_dx = nullptr;
  L->stg_dw = nullptr;
  L->stg_tokens = 0;
}

}  // namespace

extern "C" const char* mst_status_string(mst_status_t st) {
  switch (st) {
    case MST_OK: return "ok";
    case MST_ERR_INVALID_ARG: return "invalid argument";
    case MST_ERR_SHAPE: return "shape or leading dimension out of range";
    case MST_ERR_DTYPE: return "unsupported dtype";
    case MST_ERR_CAPACITY: return "nnz exceeds the layer's capacity";
    case MST_ERR_INFEASIBLE: return "no feasible prune/grow counts";
    case MST_ERR_NONFINITE: return "non-finite selection key";
    case MST_ERR_CORRUPT: return "sparse structure is corrupt";
    case MST_ERR_CUDA: return "CUDA runtime error";
    case MST_ERR_NOT_PACKED: return "layer has no structure yet";
  }
  return "unknown status";
}

extern "C" mst_status_t mst_layer_create(mst_layer_t** out, int32_t layer_id, int32_t O, int32_t I, mst_dtype_t dtype,
                                         int64_t cap) {
  if (!out) return MST_ERR_INVALID_ARG;
  *out = nullptr;
  if (dtype != MST_F32 && dtype != MST_BF16) return MST_ERR_DTYPE;
  if (O < 1 || I < 1 || O > 65535 || I > 65535) return MST_ERR_SHAPE;
  const int64_t N = (int64_t)O * I;
  if (cap < 1 || cap > N) return MST_ERR_CAPACITY;
  mst_layer* L = new (std::nothrow) mst_layer();
  if (!L) return MST_ERR_INVALID_ARG;
  L->layer_id = layer_id;
  L->O = O;
  L->I = I;
  L->dtype = dtype;
  L->cap = cap;
  L->N = N;
  L->wpr = (I + 31) / 32;
  L->wpc = (O + 31) / 32;
  L->nwords = (int64_t)O * L->wpr;
  L->nwordsT = (int64_t)I * L->wpc;
  L->nnz = -1;
  L->cur = 0;
  L->version = 0;
  L->track_values = 0;
  L->values_epoch = 0;
  L->dense_version = L->dense_epoch = -1;
  const int64_t wmax = L->nwords > L->nwordsT ? L->nwords : L->nwordsT;
  const size_t es = mst_elem_size(dtype);

  Carver cv;
  size_t o_bits[2], o_wscan[2], o_rowptr[2], o_col[2], o_vals[2];
  for (int s = 0; s < 2; ++s) {
    o_bits[s] = cv.take(4 * (size_t)L->nwords);
    o_wscan[s] = cv.take(4 * (size_t)(L->nwords + 1));
    o_rowptr[s] = cv.take(4 * (size_t)(O + 1));
    o_col[s] = cv.take(2 * (size_t)cap);
    o_vals[s] = cv.take(es * (size_t)cap);
  }
  const size_t o_pruned = cv.take(4 * (size_t)L->nwords);
  const size_t o_grad = cv.take(4 * (size_t)L->nwords);
  const size_t o_rand = cv.take(4 * (size_t)L->nwords);
  const size_t o_cnt = cv.take(4 * (size_t)(wmax + 1));
  const size_t o_scan = cv.take(4 * (size_t)(wmax + 1));
  const size_t o_bsum = cv.take(4 * (size_t)(mst_scan_block_sums_len(wmax) + 1024));
  const size_t o_hist = cv.take(4 * (size_t)MST_SELECT_BINS * 2 * 3);
  int64_t rand_cap = N / 64;
  if (rand_cap < 1024) rand_cap = 1024;
  if (rand_cap > 32768) rand_cap = 32768;
  const size_t o_rlist = cv.take(16 * (size_t)rand_cap);
  const size_t o_rctr = cv.take(16);
  const size_t o_sel = cv.take(sizeof(mst_select_state));
  const size_t o_flags = cv.take(4 * 4);
  const size_t o_counter = cv.take(4);

  unsigned char* base = nullptr;
  if (cudaMalloc((void**)&base, cv.off) != cudaSuccess) {
    delete L;
    return MST_ERR_CUDA;
  }
  if (cudaMemset(base, 0, cv.off) != cudaSuccess) {
    cudaFree(base);
    delete L;
    return MST_ERR_CUDA;
  }
  for (int s = 0; s < 2; ++s) {
    L->bits[s] = (uint32_t*)(base + o_bits[s]);
    L->wscan[s] = (int32_t*)(base + o_wscan[s]);
    L->row_ptr[s] = (int32_t*)(base + o_rowptr[s]);
    L->col_idx[s] = (uint16_t*)(base + o_col[s]);
    L->vals[s] = (void*)(base + o_vals[s]);
  }
  L->csc_base = nullptr;
  L->bitsT = nullptr;
  L->wscanT = nullptr;
  L->col_ptr = nullptr;
  L->row_idx = nullptr;
  L->perm = nullptr;
  L->pruned_bits = (uint32_t*)(base + o_pruned);
  L->grad_bits = (uint32_t*)(base + o_grad);
  L->rand_bits = (uint32_t*)(base + o_rand);
  L->word_cnt = (int32_t*)(base + o_cnt);
  L->word_scan = (int32_t*)(base + o_scan);
  L->block_sums = (int32_t*)(base + o_bsum);
  L->hist = (unsigned int*)(base + o_hist);
  L->rand_list = (unsigned long long*)(base + o_rlist);
  L->rand_ctr = (unsigned long long*)(base + o_rctr);
  L->rand_cap = (int)rand_cap;
  L->scratch_clean = 1;   // the allocation was cleared above
  L->longest_row_version = -1;
  L->sel = (mst_select_state*)(base + o_sel);
  L->flags = (int32_t*)(base + o_flags);
  L->counter = (unsigned int*)(base + o_counter);
  L->dense_w = nullptr;
  L->csc_valid = 0;
  L->path = MST_PATH_AUTO;
  L->stg_x = L->stg_dy = L->stg_y = L->stg_dx = nullptr;
  L->stg_dw = nullptr;
  L->stg_tokens = 0;
  L->async_ready = 0;
  *out = L;
  return MST_OK;
}

// The CSC view (column pointers, row indices, CSC->CSR permutation, transposed bit mask and its scan) and the dense
// bf16 image live in allocations of their own, made when a call first needs them: a layer that stays on the tensor
// path never allocates the view, a layer on the CUDA-core or structured-sparse path never allocates the image.
mst_status_t mst_alloc_csc(mst_layer* L) {
  if (L->csc_base) return MST_OK;
  Carver cv;
  const size_t o_bitsT = cv.take(4 * (size_t)L->nwordsT);
  const size_t o_wscanT = cv.take(4 * (size_t)(L->nwordsT + 1));
  const size_t o_colptr = cv.take(4 * (size_t)(L->I + 1));
  const size_t o_rowidx = cv.take(2 * (size_t)L->cap);
  const size_t o_perm = cv.take(4 * (size_t)L->cap);
  unsigned char* base = nullptr;
  MST_CUDA_TRY(cudaMalloc((void**)&base, cv.off));
  L->csc_base = base;
  L->bitsT = (uint32_t*)(base + o_bitsT);
  L->wscanT = (int32_t*)(base + o_wscanT);
  L->col_ptr = (int32_t*)(base + o_colptr);
  L->row_idx = (uint16_t*)(base + o_rowidx);
  L->perm = (int32_t*)(base + o_perm);
  L->csc_valid = 0;
  return MST_OK;
}

mst_status_t mst_alloc_dense(mst_layer* L) {
  if (L->dense_w || L->dtype != MST_BF16) return MST_OK;
  MST_CUDA_TRY(cudaMalloc((void**)&L->dense_w, 2 * (size_t)L->N));
  L->dense_version = L->dense_epoch = -1;
  return MST_OK;
}

extern "C" mst_status_t mst_layer_destroy(mst_layer_t* L) {
  if (!L) return MST_OK;
  if (L->async_ready) {
    cudaStreamSynchronize(L->s_in);
    cudaStreamSynchronize(L->s_out);
    cudaStreamDestroy(L->s_in);
    cudaStreamDestroy(L->s_out);
    cudaEventDestroy(L->ev_in);
    cudaEventDestroy(L->ev_compute);
    cudaEventDestroy(L->ev_out);
  }
  free_staging(L);
  mst_sp24_free(L);
  cudaFree(L->csc_base);
  cudaFree(L->dense_w);
  cudaFree(L->bits[0]);  // base of the main allocation
  delete L;
  return MST_OK;
}

extern "C" mst_status_t mst_set_compute_path(mst_layer_t* L, mst_compute_path_t path) {
  if (!L || path < MST_PATH_AUTO || path > MST_PATH_SPARSE_TC) return MST_ERR_INVALID_ARG;
  L->path = path;
  return MST_OK;
}

// On B200 the dense-tile tensor-core kernels beat the CUDA-core sparse kernels at every density the method visits
// (measured down to 2 %: the tensor pipe is about 18x the fp32 FMA pipe and the sparse kernels pay a staging cost
// that does not shrink with nnz), so AUTO means tensor cores whenever the layer is bf16; the launchers fall back to
// the CUDA-core kernels when an operand is not 16-byte aligned.
bool mst_use_tensor_path(const mst_layer* L) {
  if (L->dtype != MST_BF16 || L->path == MST_PATH_CUDA_CORE) return false;
  return true;
}

// Forward and input gradient on the structured-sparse instruction: on request, or under AUTO up to the density where
// it was measured faster than dense tiles.
bool mst_use_sparse_tc_path(const mst_layer* L) {
  if (L->dtype != MST_BF16 || L->nnz < 0) return false;
  if (L->path == MST_PATH_SPARSE_TC) return true;
  return false;
}

extern "C" mst_status_t mst_track_values(mst_layer_t* L, int32_t enable) {
  if (!L) return MST_ERR_INVALID_ARG;
  L->track_values = enable ? 1 : 0;
  L->dense_version = L->dense_epoch = -1;
  for (int d = 0; d < 2; ++d) L->sp[d].values_epoch = -1;
  return MST_OK;
}

extern "C" mst_status_t mst_values_changed(mst_layer_t* L) {
  if (!L) return MST_ERR_INVALID_ARG;
  ++L->values_epoch;
  return MST_OK;
}

extern "C" mst_status_t mst_layer_path_in_use(const mst_layer_t* L, mst_compute_path_t* path) {
  if (!L || !path) return MST_ERR_INVALID_ARG;
  if (mst_use_sparse_tc_path(L) && L->nnz / 2 <= L->N / 8) *path = MST_PATH_SPARSE_TC;
  else if (mst_use_tensor_path(L)) *path = MST_PATH_TENSOR_CORE;
  else *path = MST_PATH_CUDA_CORE;
  return MST_OK;
}

extern "C" mst_status_t mst_launch_count(int64_t* count) {
  if (!count) return MST_ERR_INVALID_ARG;
  *count = (int64_t)g_mst_launches.load(std::memory_order_relaxed);
  return MST_OK;
}

extern "C" mst_status_t mst_layer_nnz(const mst_layer_t* L, int64_t* nnz) {
  if (!L || !nnz) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  *nnz = L->nnz;
  return MST_OK;
}

extern "C" mst_status_t mst_values(mst_layer_t* L, void** vals, int64_t* nnz) {
  if (!L || !vals) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  *vals = L->vals[L->cur];
  if (nnz) *nnz = L->nnz;
  return MST_OK;
}

extern "C" mst_status_t mst_layer_step_host_async(mst_layer_t* L, const void* X_host, const void* dY_host, int64_t T,
                                                  void* Y_host, void* dX_host, float* dW_host, mst_stream_t stream) {
  if (!L || T < 0 || (T > 0 && (!X_host || !dY_host))) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t es = mst_elem_size(L->dtype);
  if (!L->async_ready) {
    MST_CUDA_TRY(cudaStreamCreateWithFlags(&L->s_in, cudaStreamNonBlocking));
    MST_CUDA_TRY(cudaStreamCreateWithFlags(&L->s_out, cudaStreamNonBlocking));
    MST_CUDA_TRY(cudaEventCreateWithFlags(&L->ev_in, cudaEventDisableTiming));
    MST_CUDA_TRY(cudaEventCreateWithFlags(&L->ev_compute, cudaEventDisableTiming));
    MST_CUDA_TRY(cudaEventCreateWithFlags(&L->ev_out, cudaEventDisableTiming));
    L->async_ready = 1;
  }
  if (T > L->stg_tokens || !L->stg_dw) {
    MST_CUDA_TRY(cudaStreamSynchronize(s));
    MST_CUDA_TRY(cudaStreamSynchronize(L->s_in));
    MST_CUDA_TRY(cudaStreamSynchronize(L->s_out));
    free_staging(L);
    const int64_t Ta = T > 0 ? T : 1;
    MST_CUDA_TRY(cudaMalloc(&L->stg_x, es * Ta * L->I));
    MST_CUDA_TRY(cudaMalloc(&L->stg_dy, es * Ta * L->O));
    MST_CUDA_TRY(cudaMalloc(&L->stg_y, es * Ta * L->O));
    MST_CUDA_TRY(cudaMalloc(&L->stg_dx, es * Ta * L->I));
    MST_CUDA_TRY(cudaMalloc((void**)&L->stg_dw, sizeof(float) * L->cap));
    L->stg_tokens = Ta;
  }
  // Inputs travel on the layer's copy-in stream as soon as the previous step's kernels have read the input staging
  // buffers; its results may still be on their way out (the two directions of the link work at the same time).
  MST_CUDA_TRY(cudaStreamWaitEvent(L->s_in, L->ev_compute, 0));
  if (T > 0) {
    MST_CUDA_TRY(cudaMemcpyAsync(L->stg_x, X_host, es * T * L->I, cudaMemcpyHostToDevice, L->s_in));
    MST_CUDA_TRY(cudaMemcpyAsync(L->stg_dy, dY_host, es * T * L->O, cudaMemcpyHostToDevice, L->s_in));
  }
  MST_CUDA_TRY(cudaEventRecord(L->ev_in, L->s_in));
  MST_CUDA_TRY(cudaStreamWaitEvent(s, L->ev_in, 0));
  MST_CUDA_TRY(cudaStreamWaitEvent(s, L->ev_out, 0));  // the previous step's results have left the output staging buffers
  MST_TRY(mst_launch_spmm(L, false, L->stg_x, L->I, T, L->stg_y, L->O, s));
  MST_TRY(mst_launch_spmm(L, true, L->stg_dy, L->O, T, L->stg_dx, L->I, s));
  MST_TRY(mst_launch_sddmm(L, L->stg_dy, L->O, L->stg_x, L->I, T, L->stg_dw, s));
  MST_CUDA_TRY(cudaEventRecord(L->ev_compute, s));
  // results travel back on the copy-out stream while the caller's stream goes on with the next layer
  MST_CUDA_TRY(cudaStreamWaitEvent(L->s_out, L->ev_compute, 0));
  if (T > 0 && Y_host) MST_CUDA_TRY(cudaMemcpyAsync(Y_host, L->stg_y, es * T * L->O, cudaMemcpyDeviceToHost, L->s_out));
  if (T > 0 && dX_host) MST_CUDA_TRY(cudaMemcpyAsync(dX_host, L->stg_dx, es * T * L->I, cudaMemcpyDeviceToHost, L->s_out));
  if (dW_host && L->nnz > 0)
    MST_CUDA_TRY(cudaMemcpyAsync(dW_host, L->stg_dw, sizeof(float) * L->nnz, cudaMemcpyDeviceToHost, L->s_out));
  MST_CUDA_TRY(cudaEventRecord(L->ev_out, L->s_out));
  return MST_OK;
}

extern "C" mst_status_t mst_layer_step_host_wait(mst_layer_t* L) {
  if (!L) return MST_ERR_INVALID_ARG;
  if (!L->async_ready) return MST_OK;
  MST_CUDA_TRY(cudaEventSynchronize(L->ev_out));
  return MST_OK;
}

extern "C" mst_status_t mst_layer_step_host(mst_layer_t* L, const void* X_host, const void* dY_host, int64_t T,
                                            void* Y_host, void* dX_host, float* dW_host, mst_stream_t stream) {
  MST_TRY(mst_layer_step_host_async(L, X_host, dY_host, T, Y_host, dX_host, dW_host, stream));
  MST_TRY(mst_layer_step_host_wait(L));
  MST_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
  return MST_OK;
}
