// Internal declarations shared by the translation units of libmst (not part of the public ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <cstdio>
#include <cstdlib>

#include "mst.h"
#include "mst_tc_sparse.cuh"

// With MST_DEBUG set in the environment a failing CUDA call is named on stderr before MST_ERR_CUDA is returned.
inline void mst_report_cuda_error(cudaError_t e, const char* what, const char* file, int line) {
  if (getenv("MST_DEBUG")) fprintf(stderr, "libmst: %s failed at %s:%d: %s\n", what, file, line, cudaGetErrorString(e));
}
#define MST_CUDA_TRY(expr)                                        \
  do {                                                            \
    cudaError_t e__ = (expr);                                     \
    if (e__ != cudaSuccess) {                                     \
      mst_report_cuda_error(e__, #expr, __FILE__, __LINE__);      \
      return MST_ERR_CUDA;                                        \
    }                                                             \
  } while (0)

// kernels enqueued by the library since it was loaded (mst_launch_count)
extern std::atomic<long long> g_mst_launches;
#define MST_COUNT_LAUNCH() ((void)g_mst_launches.fetch_add(1, std::memory_order_relaxed))

// Programmatic dependent launch.  A kernel started with mst_launch_overlapped may become resident and run its set-up
// (barrier initialisation, tensor-memory allocation, descriptor fetch) while its predecessor in the stream drains; it
// executes mst_grid_dependency_wait() before it reads or writes global memory (a no-op for a normal launch), and
// mst_grid_launch_dependents() as early as it likes to let its own successor do the same.  MST_PDL=0 turns the
// launch attribute off.
#ifdef __CUDACC__
__device__ __forceinline__ void mst_grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void mst_grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

inline int mst_pdl_enabled() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("MST_PDL");
    v = (e && e[0] == '0') ? 0 : 1;
  }
  return v;
}

template <typename... KArgs, typename... Args>
inline cudaError_t mst_launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                         Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = mst_pdl_enabled();
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  g_mst_launches.fetch_add(1, std::memory_order_relaxed);
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

#define MST_TRY(expr)                   \
  do {                                  \
    mst_status_t s__ = (expr);          \
    if (s__ != MST_OK) return s__;      \
  } while (0)

// Device-side error flag bits (sticky, in handle-owned memory).
enum { MST_FLAG_NONFINITE = 1, MST_FLAG_CORRUPT = 2 };

// Scratch of one radix-select run (device resident; nothing comes back to the host).
struct mst_select_state {
  unsigned long long prefix;  // digits fixed so far (left-aligned into the low bits as they are found)
  long long k;                // how many more entries to take among those matching the prefix
  unsigned long long tau;     // final threshold key
  long long rem;              // entries equal to tau to take, in index order
  int need_rank;              // 1 when more entries equal tau than are taken (their index order then decides)
  int pad;                    // "done": set when an early pass already fixed the threshold (later passes return at once)
};

struct mst_layer {
  int32_t layer_id, O, I;
  mst_dtype_t dtype;
  int64_t cap, N;
  int32_t wpr;        // 32-bit mask words per row      = ceil(I/32)
  int32_t wpc;        // mask words per transposed row  = ceil(O/32)
  int64_t nwords;     // O * wpr
  int64_t nwordsT;    // I * wpc
  int64_t nnz;        // host copy, -1 = not packed
  int cur;            // which of the two buffer sets is live
  int64_t version;    // bumped whenever the mask changes (pack, accepted topology update)
  // Value tracking (mst_track_values): the caller announces in-place changes of the stored values with
  // mst_values_changed; operands derived from the values (dense image, compressed 2:4 operand) are then rebuilt only
  // when the mask or the values have changed since they were built.  Off: rebuilt at every product call.
  int track_values;
  int64_t values_epoch;
  mutable int64_t dense_version, dense_epoch;   // what the dense image was built from (-1: nothing)

  // live structure is set [cur]; a topology update builds set [cur^1] and flips
  uint32_t* bits[2];     // [nwords]    bit (o, i) at word o*wpr + i/32, bit i%32
  int32_t* wscan[2];     // [nwords+1]  exclusive scan of popc(bits): CSR position of a word's first entry
  int32_t* row_ptr[2];   // [O+1]
  uint16_t* col_idx[2];  // [cap]
  void* vals[2];         // [cap] layer dtype

  // CSC view of the live structure.  Built at pack; the fused update skips it for layers whose input gradient runs
  // on the tensor path (which reads the dense image, not the CSC view) and it is then rebuilt on first use.
  // Allocated on first use (mst_alloc_csc): layers that never leave the tensor path never pay for it.
  mutable int csc_valid;
  unsigned char* csc_base;  // the view's own allocation, nullptr until it is needed
  uint32_t* bitsT;       // [nwordsT]
  int32_t* wscanT;       // [nwordsT+1]
  int32_t* col_ptr;      // [I+1]
  uint16_t* row_idx;     // [cap]
  int32_t* perm;         // [cap]  CSR position of each CSC entry

  // scratch for selection and rebuild
  uint32_t* pruned_bits;  // [nwords]
  uint32_t* grad_bits;    // [nwords]
  uint32_t* rand_bits;    // [nwords]
  int32_t* word_cnt;      // [max(nwords, nwordsT)+1]
  int32_t* word_scan;     // [max(nwords, nwordsT)+1]
  int32_t* block_sums;    // scan partials
  unsigned int* hist;     // [3][2 * MST_SELECT_BINS]: rotating global histograms of the radix select (two selections side by side)
  unsigned long long* rand_list;  // [rand_cap][2]: hash key and flat index of the random-growth candidates inside the bracket
  unsigned long long* rand_ctr;   // [2]: candidates below the bracket, list length
  int rand_cap;
  int scratch_clean;      // hist and rand_ctr are known to be zero (the fused update kernel leaves them so)
  mst_select_state* sel;  // [1]
  int32_t* flags;         // [4]: error bits, max row nnz of the last update, longest row (CUDA-core forward), spare
  mutable int64_t longest_row_version;  // structure version flags[2] belongs to
  unsigned int* counter;  // [1] block-completion counter

  // dense bf16 image of W.M for the tensor-core path (bf16 layers only): [O x I]; the input gradient reads it as an
  // MN-major operand, so no transposed copy is kept.  Allocated on first use (mst_alloc_dense).
  uint16_t* dense_w;
  int path;  // mst_compute_path_t
  // 2:4 split of W.M (forward) and of its transpose (input gradient) for the structured-sparse tensor-core path;
  // allocated on first use
  mst_sp24 sp[2];

  // host staging for mst_layer_step_host
  void *stg_x, *stg_dy, *stg_y, *stg_dx;
  float* stg_dw;
  int64_t stg_tokens;
  // copy streams and events of the asynchronous host step (created on first use)
  cudaStream_t s_in, s_out;
  cudaEvent_t ev_in, ev_compute, ev_out;
  int async_ready;
};

static inline size_t mst_elem_size(mst_dtype_t d) { return d == MST_F32 ? 4 : 2; }

// structure (mst_structure.cu)
mst_status_t mst_scan_i32(const int32_t* in, int32_t* out, int64_t n, int32_t* block_sums, cudaStream_t s);
int64_t mst_scan_block_sums_len(int64_t n);
// same scan, but every block returns at once when *enabled (device memory) is 0
mst_status_t mst_scan_i32_if(const int32_t* in, int32_t* out, int64_t n, int32_t* block_sums, const int* enabled,
                             cudaStream_t s);
mst_status_t mst_rebuild_from_bits(mst_layer* L, int set, const void* dense_W, int64_t ldw, int old_set, cudaStream_t s);
mst_status_t mst_alloc_csc(mst_layer* L);     // no-op when the view's arrays exist
mst_status_t mst_alloc_dense(mst_layer* L);   // no-op when the dense image exists
mst_status_t mst_build_csc(mst_layer* L, cudaStream_t s);
mst_status_t mst_ensure_csc(const mst_layer* L, cudaStream_t s);  // builds the CSC view if it is stale
mst_status_t mst_combine_update_bits(mst_layer* L, int new_set, cudaStream_t s);
mst_status_t mst_densify(const mst_layer* L, cudaStream_t s, const uint16_t** image);
// strided attention forward on warp-level products (mst_attention_fwd_mma.cu); the caller has checked pointers and
// leading dimensions
mst_status_t mst_attention_fwd_mma(const void* Q, const void* K, const void* V, int64_t ld, int32_t batch, int32_t seq_len,
                                   int32_t heads, int32_t stride, void* Out, int64_t ldo, float* lse, cudaStream_t s);
bool mst_use_tensor_path(const mst_layer* L);
bool mst_use_sparse_tc_path(const mst_layer* L);

// sticky error word of the CUDA-core SpMM's bounded waits (mst_spmm.cu)
mst_status_t mst_spmm_error_flags(int32_t* flags);
mst_status_t mst_sddmm_error_flags(int32_t* flags);
// sticky error word of the attention kernel's bounded waits (mst_attention.cu)
mst_status_t mst_attention_error_flags(int32_t* flags);

// bins of one radix-select pass (digit width MST_SELECT_RADIX_BITS)
constexpr int MST_SELECT_RADIX_BITS = 11;
constexpr int MST_SELECT_BINS = 1 << MST_SELECT_RADIX_BITS;

// kernels' launchers
// act / pre / ldpre: element-wise step fused behind the product (see mst_tc_gemm.cuh); act = 0 for the plain product
mst_status_t mst_launch_spmm(const mst_layer* L, bool transpose, const void* in, int64_t ldin, int64_t T, void* out,
                             int64_t ldout, cudaStream_t s, int act = 0, void* pre = nullptr, int64_t ldpre = 0);
mst_status_t mst_launch_sddmm(const mst_layer* L, const void* dY, int64_t lddy, const void* X, int64_t ldx, int64_t T,
                              float* dW, cudaStream_t s);
