// Mixed-Growing topology update (Algorithm 1) on the device.
//
// The three selections of the algorithm (prune by smallest |w|, grow by largest |g|, grow at random) are the same
// primitive: take the k smallest keys of a candidate set, ties broken by the smaller flat index.  Each is done by a
// most-significant-digit radix select (11 bits per pass) that leaves a threshold key tau and the number `rem` of
// entries equal to tau still to take; a popcount + exclusive scan over the mask words then ranks the entries equal to
// tau in flat-index order and the first `rem` of them are taken.  Results are bit masks over the flat index space, so
// the mask rewrite is three bitwise operations per word and the CSR rebuild is the popcount/scan/fill of
// mst_structure.cu.  Integer keys, integer atomics only: the outcome is deterministic and bit-exact.
//
// Work layout: one warp per 32-bit mask word, lane = column inside the word, so reads of G and of the value array are
// coalesced.  Three forms, all with the same results:
//  - kernel per phase (run_select): the last block to finish a histogram pass picks the digit;
//  - one cooperative kernel, one selection after the other (fused_select);
//  - one cooperative kernel with the prune and the gradient selection side by side and the random growth by bracket
//    (fused_dual_update), the default whenever just-pruned links may not be regrown: keys of a block's slice in
//    shared memory, gradients copied there asynchronously, work on the few active entries of a word done by one
//    thread per word, the random threshold found among the few candidates whose hash falls into a precomputed bracket.
// The tie ranking (count, scan) is skipped on the device when the threshold key has no surplus ties.
#include <cooperative_groups.h>

#include <cmath>
#include <cstdlib>
#include <new>

#include "mst_bits.cuh"
#include "mst_internal.cuh"

namespace {

enum { MODE_PRUNE = 0, MODE_GRAD = 1, MODE_RAND = 2 };

struct SelParams {
  const uint32_t* old_bits;
  const int32_t* old_wscan;
  const void* vals;
  int bf16;
  const float* G;
  const uint32_t* pruned_bits;
  const uint32_t* grad_bits;
  int O, I, wpr, allow;
  int aligned;   // I % 32 == 0
  int low_zero;  // low key bits known to be zero in the prune keys (16 for bf16 values)
  float lambda;  // MEST prune key |w| + lambda |g| when non-zero
  int64_t nwords;
  unsigned long long stream;
};

__device__ __forceinline__ unsigned lanemask_lt() {
  unsigned m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

// SplitMix64 output function (Steele, Lea, Flood 2014)
__device__ __forceinline__ unsigned long long sm64_mix(unsigned long long z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}
constexpr unsigned long long SM64_GAMMA = 0x9E3779B97F4A7C15ULL;

template <int MODE>
struct KeyBits {
  static constexpr int value = MODE == MODE_RAND ? 64 : 32;
};
template <int MODE>
struct KeyWord {
  typedef uint32_t type;
};
template <>
struct KeyWord<MODE_RAND> {
  typedef unsigned long long type;
};

// candidate test and key of bit `lane` of word w.  nonfinite is set when a magnitude key is Inf/NaN.
template <int MODE>
__device__ __forceinline__ bool cand_key_w(const SelParams& P, int64_t w, int lane, uint32_t old_word, int32_t old_base,
                                           uint32_t grad_word, unsigned long long& key, bool& nonfinite) {
  // flat index of this bit; when I is a multiple of 32 the mask words tile the flat index space exactly
  long long f;
  bool col_ok = true;
  if (P.aligned) {
    f = (long long)w * 32 + lane;
  } else {
    const unsigned wu = (unsigned)w, wpr = (unsigned)P.wpr;  // nwords < 2^31
    const int o = (int)(wu / wpr), c = (int)(wu - (unsigned)o * wpr) * 32 + lane;
    col_ok = c < P.I;
    f = (long long)o * P.I + c;
  }
  nonfinite = false;
  key = 0;
  if (MODE == MODE_PRUNE) {
    const uint32_t word = old_word;
    if (!((word >> lane) & 1u)) return false;
    const int32_t pos = old_base + __popc(word & lanemask_lt());
    uint32_t k;
    if (P.bf16)
      k = ((uint32_t)(((const uint16_t*)P.vals)[pos] & 0x7FFFu)) << 16;
    else
      k = ((const uint32_t*)P.vals)[pos] & 0x7FFFFFFFu;
    if (P.lambda != 0.f) {  // MEST criterion, fp32 with one rounding per operation (never contracted to an FMA)
      const float g = fabsf(P.G[f]);
      k = __float_as_uint(__fadd_rn(__uint_as_float(k), __fmul_rn(P.lambda, g))) & 0x7FFFFFFFu;
    }
    nonfinite = k >= 0x7F800000u;
    key = k;
    return true;
  } else if (MODE == MODE_GRAD) {
    uint32_t word = ~old_word;
    if (P.allow) word |= P.pruned_bits[w];
    if (!col_ok || !((word >> lane) & 1u)) return false;
    const uint32_t k = __float_as_uint(P.G[f]) & 0x7FFFFFFFu;
    nonfinite = k >= 0x7F800000u;
    key = 0xFFFFFFFFu - k;  // largest magnitude first
    return true;
  } else {
    const uint32_t word = ~old_word & ~grad_word;
    if (!col_ok || !((word >> lane) & 1u)) return false;
    key = sm64_mix(P.stream + SM64_GAMMA * ((unsigned long long)f + 1ULL));
    return true;
  }
}

// same, with the mask words fetched from global memory
template <int MODE>
__device__ __forceinline__ bool cand_key(const SelParams& P, int64_t w, int lane, unsigned long long& key,
                                         bool& nonfinite) {
  const uint32_t ow = P.old_bits[w];
  const int32_t ob = MODE == MODE_PRUNE ? P.old_wscan[w] : 0;
  const uint32_t gw = MODE == MODE_RAND ? P.grad_bits[w] : 0u;
  return cand_key_w<MODE>(P, w, lane, ow, ob, gw, key, nonfinite);
}

constexpr int RADIX_BITS = MST_SELECT_RADIX_BITS;
constexpr int BINS = MST_SELECT_BINS;
constexpr int HIST_THREADS = 1024;
constexpr int BINS_PER_THREAD = BINS / HIST_THREADS;

__host__ __device__ constexpr int num_passes(int key_bits) { return (key_bits + RADIX_BITS - 1) / RADIX_BITS; }
// digit `pass` (most significant first) covers key bits [pass_shift, pass_shift + pass_width)
__host__ __device__ constexpr int pass_shift(int key_bits, int pass) {
  return key_bits - RADIX_BITS * (pass + 1) > 0 ? key_bits - RADIX_BITS * (pass + 1) : 0;
}
__host__ __device__ constexpr int pass_width(int key_bits, int pass) {
  return key_bits - RADIX_BITS * pass < RADIX_BITS ? key_bits - RADIX_BITS * pass : RADIX_BITS;
}

__global__ void select_init(mst_select_state* st, long long k, unsigned int* hist, unsigned int* counter) {
  if (threadIdx.x == 0) {
    st->prefix = 0;
    st->k = k;
    st->tau = 0;
    st->rem = 0;
    st->need_rank = 0;
    st->pad = 0;   // 'done' flag: later passes return at once
    *counter = 0;
  }
  for (int b = threadIdx.x; b < BINS; b += blockDim.x) hist[b] = 0;
}

template <int MODE>
__global__ void __launch_bounds__(HIST_THREADS) select_hist(SelParams P, int pass, mst_select_state* st, unsigned int* hist,
                                                   unsigned int* counter, int32_t* flags) {
  constexpr int KB = KeyBits<MODE>::value;
  __shared__ unsigned int sh[BINS];
  __shared__ unsigned int warp_tot[HIST_THREADS / 32];
  __shared__ bool is_last;
  if (st->pad) return;  // an earlier pass already fixed the threshold
  for (int b = threadIdx.x; b < BINS; b += HIST_THREADS) sh[b] = 0;
  __syncthreads();
  const unsigned long long prefix = st->prefix;
  const int shift = pass_shift(KB, pass);
  const unsigned dmask = (1u << pass_width(KB, pass)) - 1u;
  const int hi_shift = shift + pass_width(KB, pass);  // bits above this digit
  const int lane = threadIdx.x & 31;
  const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  bool saw_nonfinite = false;
  // four words per trip so that their dependent loads (mask word -> position -> value) overlap
  constexpr int BATCH = 4;
  for (int64_t w0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w0 < P.nwords; w0 += warps * BATCH) {
    unsigned digit[BATCH];
    bool live[BATCH];
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      const int64_t w = w0 + (int64_t)j * warps;
      unsigned long long key = 0;
      bool nf = false;
      const bool c = w < P.nwords && cand_key<MODE>(P, w, lane, key, nf);
      saw_nonfinite |= (c && nf);
      // entries whose higher digits differ from the prefix are out of the race
      live[j] = c && (pass == 0 || (key >> hi_shift) == prefix);
      digit[j] = live[j] ? (unsigned)((key >> shift) & dmask) : (unsigned)BINS;
    }
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      if (live[j]) atomicAdd(&sh[digit[j]], 1u);
    }
  }
  if (pass == 0 && saw_nonfinite) atomicOr(&flags[0], MST_FLAG_NONFINITE);
  __syncthreads();
  for (int b = threadIdx.x; b < BINS; b += HIST_THREADS)
    if (sh[b]) atomicAdd(&hist[b], sh[b]);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(counter, 1u) == gridDim.x - 1);
  __syncthreads();
  if (!is_last) return;
  // last block to finish: every other block's contribution is visible; pick the digit that holds the k-th key
  __threadfence();
  unsigned int mine[BINS_PER_THREAD];
  unsigned int tsum = 0;
#pragma unroll
  for (int j = 0; j < BINS_PER_THREAD; ++j) {
    const int b = threadIdx.x * BINS_PER_THREAD + j;
    mine[j] = atomicAdd(&hist[b], 0u);
    hist[b] = 0;  // ready for the next pass
    tsum += mine[j];
  }
  // exclusive prefix of the per-thread sums over the block
  unsigned int incl = tsum;
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) warp_tot[threadIdx.x >> 5] = incl;
  __syncthreads();
  unsigned int before = incl - tsum;
  for (int wv = 0; wv < (int)(threadIdx.x >> 5); ++wv) before += warp_tot[wv];
  const long long k = st->k;
  __syncthreads();  // everyone has read st->k before the owner rewrites it
  const bool owner = (long long)before < k && k <= (long long)before + (long long)tsum;
  if (owner) {
    long long cum = before;
    int bin = 0;
#pragma unroll
    for (int j = 0; j < BINS_PER_THREAD; ++j) {
      if (cum + (long long)mine[j] >= k) { bin = j; break; }
      cum += mine[j];
    }
    const unsigned long long np = (prefix << pass_width(KB, pass)) | (unsigned long long)(threadIdx.x * BINS_PER_THREAD + bin);
    st->prefix = np;
    st->k = k - cum;
    if (shift == 0) {
      st->tau = np;
      st->rem = k - cum;
      st->need_rank = ((long long)mine[bin] > k - cum) ? 1 : 0;  // ties at the threshold beyond what is taken
    } else if ((long long)mine[bin] == k - cum) {
      // every key that shares this prefix is taken: the lower digits cannot matter, stop here
      st->tau = (np << shift) | ((1ULL << shift) - 1ULL);
      st->rem = k - cum;
      st->need_rank = 0;
      st->pad = 1;
    }
  }
  if (threadIdx.x == HIST_THREADS - 1) {
    const long long total = (long long)before + (long long)tsum;
    if (total < k) atomicOr(&flags[0], MST_FLAG_CORRUPT);  // fewer candidates than requested: ruled out by the host counts
    *counter = 0;
  }
}

// cnt[w] = number of candidates in word w whose key equals tau (skipped when no tie has to be ranked)
template <int MODE>
__global__ void __launch_bounds__(256) select_count_equal(SelParams P, const mst_select_state* st,
                                                          int32_t* __restrict__ cnt) {
  if (!st->need_rank) return;
  const unsigned long long tau = st->tau;
  const int lane = threadIdx.x & 31;
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (w >= P.nwords) return;
  unsigned long long key;
  bool nf;
  const bool c = cand_key<MODE>(P, w, lane, key, nf);
  const unsigned eq = __ballot_sync(0xffffffffu, c && key == tau);
  if (lane == 0) cnt[w] = __popc(eq);
}

template <int MODE>
__global__ void __launch_bounds__(256) select_mark(SelParams P, const mst_select_state* st,
                                                   const int32_t* __restrict__ eq_scan, uint32_t* __restrict__ out) {
  const unsigned long long tau = st->tau;
  const long long rem = st->rem;
  const bool need_rank = st->need_rank != 0;
  const int lane = threadIdx.x & 31;
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (w >= P.nwords) return;
  unsigned long long key;
  bool nf;
  const bool c = cand_key<MODE>(P, w, lane, key, nf);
  const bool iseq = c && key == tau;
  const unsigned eq = __ballot_sync(0xffffffffu, iseq);
  // without ties beyond the quota every entry equal to tau is taken; otherwise the first `rem` in index order
  const long long rank = need_rank ? (long long)eq_scan[w] + __popc(eq & lanemask_lt()) : -1;
  const bool take = c && (key < tau || (iseq && rank < rem));
  const unsigned bits = __ballot_sync(0xffffffffu, take);
  if (lane == 0) out[w] = bits;
}

__global__ void max_row_nnz(const int32_t* __restrict__ row_ptr, int O, int32_t* flags) {
  const int o = blockIdx.x * blockDim.x + threadIdx.x;
  if (o < O) atomicMax(&flags[1], row_ptr[o + 1] - row_ptr[o]);
}

template <int MODE>
mst_status_t run_select(mst_layer* L, const SelParams& P, int64_t k, uint32_t* out_bits, cudaStream_t s) {
  if (k <= 0) {
    MST_CUDA_TRY(cudaMemsetAsync(out_bits, 0, sizeof(uint32_t) * L->nwords, s));
    return MST_OK;
  }
  constexpr int passes = num_passes(KeyBits<MODE>::value);
  select_init<<<1, 256, 0, s>>>(L->sel, (long long)k, L->hist, L->counter); MST_COUNT_LAUNCH();
  int64_t blocks = (L->nwords * 32 + HIST_THREADS - 1) / HIST_THREADS;
  if (blocks > 2 * 148) blocks = 2 * 148;  // all SMs fully occupied; each block ends with one global add per non-empty bin
  for (int p = 0; p < passes; ++p)
    { select_hist<MODE><<<(unsigned)blocks, HIST_THREADS, 0, s>>>(P, p, L->sel, L->hist, L->counter, L->flags); MST_COUNT_LAUNCH(); }
  const unsigned wgrid = (unsigned)((L->nwords * 32 + 255) / 256);
  select_count_equal<MODE><<<wgrid, 256, 0, s>>>(P, L->sel, L->word_cnt); MST_COUNT_LAUNCH();
  MST_TRY(mst_scan_i32_if(L->word_cnt, L->word_scan, L->nwords, L->block_sums, &L->sel->need_rank, s));
  select_mark<MODE><<<wgrid, 256, 0, s>>>(P, L->sel, L->word_scan, out_bits); MST_COUNT_LAUNCH();
  MST_CUDA_TRY(cudaGetLastError());
  return MST_OK;
}

// ------------------------------------------------------------------------------------------------ fused update
// The whole update as ONE cooperative kernel: the phases above (histogram passes, digit picks, tie ranking, marking,
// mask rewrite, scans, CSR and CSC fill) separated by grid-wide barriers instead of kernel boundaries.  Every block
// owns one contiguous slice of the mask words for all word-wise phases, so that only the histogram -> pick steps, the
// scans and the transpose need a barrier.  Every block computes each digit pick itself from the global histogram
// (three rotating histogram buffers: the one for pass p+2 is cleared after the barrier of pass p).
namespace cg = cooperative_groups;

#ifdef MST_UPD_PROFILE
// phase stamps of block 0 of the last fused update (SM clock), read back through mst_update_profile
__device__ long long g_upd_stamps[64];
__device__ int g_upd_nstamps;
#define UPD_STAMP(id)                                                      \
  do {                                                                     \
    if (blockIdx.x == 0 && threadIdx.x == 0) {                             \
      const int at_ = g_upd_nstamps;                                       \
      if (at_ < 31) {                                                      \
        g_upd_stamps[2 * at_] = (id);                                      \
        g_upd_stamps[2 * at_ + 1] = clock64();                             \
        g_upd_nstamps = at_ + 1;                                           \
      }                                                                    \
    }                                                                      \
  } while (0)
#else
#define UPD_STAMP(id) do { } while (0)
#endif

constexpr int FUSED_THREADS = 512;
constexpr int FUSED_WARPS = FUSED_THREADS / 32;
constexpr int FUSED_BPT = BINS / FUSED_THREADS;  // histogram bins per thread in the pick

struct FusedParams {
  SelParams sel;
  long long n_prune, n_grad, n_rand;
  uint32_t *pruned_bits, *grad_bits, *rand_bits, *new_bits;
  int32_t *cnt, *scan, *bsums;
  unsigned int* hist;  // [3][HSTRIDE], all zero at launch and again at exit
  int32_t* flags;
  int32_t *new_wscan, *new_row_ptr;
  uint16_t* new_col;
  void* new_vals;
  uint32_t* bitsT;
  int32_t *wscanT, *col_ptr;
  uint16_t* row_idx;
  int32_t* perm;
  int wpc;
  int64_t nwordsT;
  int build_csc;  // 0: leave the CSC view stale (the layer's input gradient reads the dense image instead)
  int smem_keys;  // 1: the launch carries shared memory for the key cache (slices too large for the registers)
  int dual;       // 1: prune and gradient selections run side by side (their candidate sets are disjoint)
  int g_bulk;     // 1: a slice's gradients are one contiguous, 16-byte aligned run (mask words tile the flat index space)
  // random growth by bracket: hash keys are uniform, so the n_rand-th smallest lies in [rand_lo, rand_hi) with
  // overwhelming probability; the candidates inside are listed and the threshold is found among them
  int rand_bracket;
  int rand_cap;                    // entries the list holds
  unsigned long long rand_lo, rand_hi;
  unsigned long long* rand_list;   // [rand_cap][2]: key, flat index
  unsigned long long* rand_ctr;    // [2]: candidates below rand_lo, list length; zero at launch and again at exit
};

constexpr int HSTRIDE = 2 * BINS;   // one rotating histogram buffer: two selections side by side
struct FusedShared {
  unsigned int hist[BINS];   // side-by-side selections count in the two 16-bit halves of a bin (a slice has < 65536 entries)
  unsigned int warp_tot[FUSED_WARPS];
  int red[FUSED_WARPS];
  unsigned long long prefix, tau;
  long long k, rem;
  int need_rank, done, found;
  // two selections side by side (0: prune, 1: gradient growth)
  uint32_t d_prefix[2], d_tau[2];
  long long d_k[2], d_rem[2];
  int d_need_rank[2], d_done[2], d_found[2];
  // random growth by bracket
  unsigned long long r_tau, r_tau_f;
  long long r_rank;
  int r_ok, r_bin, r_n;
};

__device__ __forceinline__ int fused_block_sum(int v, FusedShared& sh) {
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();  // sh.red free
  if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = v;
  __syncthreads();
  int r = 0;
#pragma unroll
  for (int w = 0; w < FUSED_WARPS; ++w) r += sh.red[w];
  return r;
}

// exclusive prefix of v over the block (thread order); total = sum over the block
__device__ __forceinline__ int fused_block_excl_scan(int v, int& total, FusedShared& sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int x = v;
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  __syncthreads();
  if (lane == 31) sh.red[warp] = x;
  __syncthreads();
  int before = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < FUSED_WARPS; ++w) {
    const int t = sh.red[w];
    if (w < warp) before += t;
    tot += t;
  }
  total = tot;
  return before + x - v;
}

// out[0..n] = exclusive scan of cnt[0..n); each block scans its slice [lo, hi).  One grid barrier inside.
// The per-block partial sums of consecutive scans alternate between two areas of `bsums` (gscan counts the scans of
// this launch): a block that has left scan k may already be writing its partial sum of scan k+1 while a slower block
// still reads the partial sums of scan k, and an area is only rewritten two scans later, behind the next barrier.
__device__ int fused_grid_scan(const int32_t* cnt, int32_t* out, int64_t n, int64_t lo, int64_t hi, int32_t* bsums,
                                int& gscan, cg::grid_group& grid, FusedShared& sh) {
  bsums += (gscan & 1) * (int)gridDim.x;
  ++gscan;
  int v = 0;
  for (int64_t i = lo + threadIdx.x; i < hi; i += FUSED_THREADS) v += cnt[i];
  const int bs = fused_block_sum(v, sh);
  if (threadIdx.x == 0) bsums[blockIdx.x] = bs;
  grid.sync();
  int off = 0, tot = 0;
  for (int j = threadIdx.x; j < (int)gridDim.x; j += FUSED_THREADS) {
    const int x = __ldcg(bsums + j);
    tot += x;
    if (j < (int)blockIdx.x) off += x;
  }
  off = fused_block_sum(off, sh);
  tot = fused_block_sum(tot, sh);
  int carry = off;
  for (int64_t base = lo; base < hi; base += FUSED_THREADS) {
    const int64_t i = base + threadIdx.x;
    const int x = i < hi ? cnt[i] : 0;
    int tile_total;
    const int ex = fused_block_excl_scan(x, tile_total, sh);
    if (i < hi) out[i] = carry + ex;
    carry += tile_total;
  }
  if (threadIdx.x == 0) out[n] = tot;  // every block writes the same total: whoever reads it next in this block sees it
  __syncthreads();
  return tot;
}

// One selection inside the fused kernel.  gpass counts the histogram passes executed so far (buffer rotation).
// Words per warp whose keys may stay in registers for a whole selection (CACHED): the warp's words are fixed
// (lo + warp + j * FUSED_WARPS), so each lane loads the key of its bit of each word once and every later pass, the tie
// count and the marking sweep work from registers instead of fetching G or the values again.  For the 64-bit hash keys
// the high word is kept; the digits below bit 32 and ties on the high word recompute the hash.
constexpr int KEYS_PER_LANE = 16;
// Larger slices (up to the shared memory a block can have) keep the same key words in shared memory instead
// (CACHE_SMEM: skey[word][lane] and one candidate mask word per mask word): the first pass of a selection computes
// every key once, all later sweeps read 4 bytes of shared memory per entry instead of fetching G / the values or
// hashing again.
enum { CACHE_NONE = 0, CACHE_REGS = 1, CACHE_SMEM = 2 };

template <int MODE, int CACHE>
__device__ void fused_select(const FusedParams& F, long long k_total, uint32_t* out_bits, int64_t lo, int64_t hi,
                             int& gpass, int& gscan, cg::grid_group& grid, FusedShared& sh, const uint32_t* s_old,
                             const int32_t* s_base, uint32_t* s_grad, uint32_t* skey, uint32_t* scand) {
  constexpr bool CACHED = CACHE == CACHE_REGS;
  constexpr int KB = KeyBits<MODE>::value;
  // magnitude keys are 32 bits wide: their passes compare and shift 32-bit words, only the hashes need 64
  typedef typename KeyWord<MODE>::type K;
  constexpr int passes = num_passes(KB);
  const SelParams& P = F.sel;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (k_total <= 0) {  // uniform over the grid
    for (int64_t w = lo + threadIdx.x; w < hi; w += FUSED_THREADS) {
      out_bits[w] = 0;
      if (MODE == MODE_GRAD) s_grad[w - lo] = 0;
    }
    __syncthreads();
    return;
  }
  if (threadIdx.x == 0) {
    sh.prefix = 0;
    sh.k = k_total;
    sh.tau = 0;
    sh.rem = 0;
    sh.need_rank = 0;
    sh.done = 0;
  }
  __syncthreads();
  uint32_t kc[KEYS_PER_LANE];  // CACHED: key word of this lane's bit of word j; bit j of candm: it is a candidate
  uint32_t candm = 0;
  bool cache_nonfinite = false;
  if (CACHED) {
#pragma unroll
    for (int j = 0; j < KEYS_PER_LANE; ++j) {
      const int64_t w = lo + warp + (int64_t)j * FUSED_WARPS;
      kc[j] = 0;
      if (w < hi) {  // uniform over the warp
        unsigned long long key64 = 0;
        bool nf = false;
        const bool c = cand_key_w<MODE>(P, w, lane, s_old[w - lo], s_base[w - lo], s_grad[w - lo], key64, nf);
        kc[j] = MODE == MODE_RAND ? (uint32_t)(key64 >> 32) : (uint32_t)key64;
        if (c) candm |= 1u << j;
        cache_nonfinite |= (c && nf);
      }
    }
  }
  if (CACHE == CACHE_SMEM) {
    for (int64_t w = lo + warp; w < hi; w += FUSED_WARPS) {
      unsigned long long key64 = 0;
      bool nf = false;
      const bool c = cand_key_w<MODE>(P, w, lane, s_old[w - lo], s_base[w - lo], s_grad[w - lo], key64, nf);
      skey[(w - lo) * 32 + lane] = MODE == MODE_RAND ? (uint32_t)(key64 >> 32) : (uint32_t)key64;
      const unsigned cm = __ballot_sync(0xffffffffu, c);
      if (lane == 0) scand[w - lo] = cm;
      cache_nonfinite |= (c && nf);
    }
    __syncwarp();   // a warp reads back only what it wrote itself
  }
  // full key of the entry of word w in this lane (a candidate): only the hash keys hold more than the cached word
  auto word_full_key = [&](int64_t w) -> K {
    unsigned long long key64 = 0;
    bool nf = false;
    cand_key_w<MODE>(P, w, lane, s_old[w - lo], s_base[w - lo], s_grad[w - lo], key64, nf);
    return (K)key64;
  };
  // full-width key of cached entry j (a candidate): only the hash keys hold more than the cached word
  auto cached_full_key = [&](int j) -> K {
    if (MODE != MODE_RAND) return (K)kc[j];
    const int64_t w = lo + warp + (int64_t)j * FUSED_WARPS;
    unsigned long long key64 = 0;
    bool nf = false;
    cand_key_w<MODE>(P, w, lane, s_old[w - lo], s_base[w - lo], s_grad[w - lo], key64, nf);
    return (K)key64;
  };
  for (int pass = 0; pass < passes; ++pass) {
    if (sh.done) break;  // same decision in every block
    const int shift = pass_shift(KB, pass), width = pass_width(KB, pass);
    const unsigned dmask = (1u << width) - 1u;
    const int hi_shift = shift + width;
    const K prefix = (K)sh.prefix;
    const long long k = sh.k;
    unsigned int* gh = F.hist + (gpass % 3) * HSTRIDE;
    for (int b = threadIdx.x; b < BINS; b += FUSED_THREADS) sh.hist[b] = 0;
    __syncthreads();
    bool saw_nonfinite = cache_nonfinite;
    constexpr int BATCH = 8;
    if (CACHED) {
      const bool hi_word = MODE == MODE_RAND && shift >= 32;  // digit and prefix lie inside the cached high word
#pragma unroll
      for (int j = 0; j < KEYS_PER_LANE; ++j) {
        if (lo + warp + (int64_t)j * FUSED_WARPS >= hi) break;  // uniform over the warp
        const bool c = (candm >> j) & 1u;
        K key = 0;
        if (MODE != MODE_RAND) key = (K)kc[j];
        else if (hi_word) key = (K)((unsigned long long)kc[j] << 32);
        else if (c) key = cached_full_key(j);
        const bool lv = c && (pass == 0 || (K)(key >> hi_shift) == prefix);
        const unsigned dg = lv ? (unsigned)((key >> shift) & (K)dmask) : (unsigned)BINS;
        // one shared-memory atomic per live lane: grouping equal digits with a warp match first was measured slower
        if (lv) atomicAdd(&sh.hist[dg], 1u);
      }
    } else if (CACHE == CACHE_SMEM) {
      const bool hi_word = MODE == MODE_RAND && shift >= 32;
      for (int64_t w = lo + warp; w < hi; w += FUSED_WARPS) {
        const uint32_t kw = skey[(w - lo) * 32 + lane];
        bool c = (scand[w - lo] >> lane) & 1u;
        K key = 0;
        if (MODE != MODE_RAND) key = (K)kw;
        else if (hi_word) key = (K)((unsigned long long)kw << 32);
        else {
          // the digit reaches below the cached word: hash again, but only for entries whose cached word can still
          // match the prefix
          if (c && pass > 0 && hi_shift >= 32) c = (K)(((unsigned long long)kw << 32) >> hi_shift) == prefix;
          if (c) key = word_full_key(w);
        }
        const bool lv = c && (pass == 0 || (K)(key >> hi_shift) == prefix);
        if (lv) atomicAdd(&sh.hist[(unsigned)((key >> shift) & (K)dmask)], 1u);
      }
    } else
    for (int64_t w0 = lo + warp; w0 < hi; w0 += FUSED_WARPS * BATCH) {
      unsigned digit[BATCH];
      bool live[BATCH];
#pragma unroll
      for (int j = 0; j < BATCH; ++j) {
        const int64_t w = w0 + (int64_t)j * FUSED_WARPS;
        unsigned long long key64 = 0;
        bool nf = false;
        const int64_t li = w < hi ? w - lo : 0;
        const bool c = w < hi && cand_key_w<MODE>(P, w, lane, s_old[li], s_base[li], s_grad[li], key64, nf);
        const K key = (K)key64;
        saw_nonfinite |= (c && nf);
        live[j] = c && (pass == 0 || (K)(key >> hi_shift) == prefix);
        digit[j] = live[j] ? (unsigned)((key >> shift) & (K)dmask) : (unsigned)BINS;
      }
#pragma unroll
      for (int j = 0; j < BATCH; ++j) {
        if (live[j]) atomicAdd(&sh.hist[digit[j]], 1u);
      }
    }
    if (pass == 0 && saw_nonfinite) atomicOr(&F.flags[0], MST_FLAG_NONFINITE);
    __syncthreads();
    for (int b = threadIdx.x; b < BINS; b += FUSED_THREADS)
      if (sh.hist[b]) atomicAdd(&gh[b], sh.hist[b]);
    grid.sync();
    // every block picks the digit from the complete histogram
    unsigned int mine[FUSED_BPT];
    unsigned int tsum = 0;
#pragma unroll
    for (int j = 0; j < FUSED_BPT; ++j) {
      mine[j] = __ldcg(gh + threadIdx.x * FUSED_BPT + j);
      tsum += mine[j];
    }
    if (blockIdx.x == 0) {  // clear the buffer of pass gpass + 2 (last read before this barrier)
      unsigned int* gz = F.hist + ((gpass + 2) % 3) * HSTRIDE;
      for (int b = threadIdx.x; b < HSTRIDE; b += FUSED_THREADS) gz[b] = 0;
    }
    unsigned int incl = tsum;
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (threadIdx.x == 0) sh.found = 0;
    if (lane == 31) sh.warp_tot[warp] = incl;
    __syncthreads();
    unsigned int before = incl - tsum;
    for (int wv = 0; wv < warp; ++wv) before += sh.warp_tot[wv];
    const bool owner = (long long)before < k && k <= (long long)before + (long long)tsum;
    if (owner) {
      long long cum = before;
      int bin = 0;
      unsigned int bcount = 0;
      for (int j = 0; j < FUSED_BPT; ++j) {
        if (cum + (long long)mine[j] >= k) { bin = j; bcount = mine[j]; break; }
        cum += mine[j];
      }
      const unsigned long long np = (prefix << width) | (unsigned long long)(threadIdx.x * FUSED_BPT + bin);
      sh.prefix = np;
      sh.k = k - cum;
      sh.found = 1;
      if (shift == 0) {
        sh.tau = np;
        sh.rem = k - cum;
        sh.need_rank = ((long long)bcount > k - cum) ? 1 : 0;
        sh.done = 1;
      } else if ((long long)bcount == k - cum) {
        sh.tau = (np << shift) | ((1ULL << shift) - 1ULL);
        sh.rem = k - cum;
        sh.need_rank = 0;
        sh.done = 1;
      } else if (MODE == MODE_PRUNE && shift <= P.low_zero) {
        // the undecided low bits are zero in every key: the bucket is one run of equal keys
        sh.tau = np << shift;
        sh.rem = k - cum;
        sh.need_rank = 1;
        sh.done = 1;
      }
    }
    __syncthreads();
    if (!sh.found) {  // fewer candidates than requested (ruled out by the host counts): take everything
      if (threadIdx.x == 0) {
        sh.tau = ~0ULL;
        sh.rem = 0x7FFFFFFFFFFFFFFFLL;
        sh.need_rank = 0;
        sh.done = 1;
        if (blockIdx.x == 0) atomicOr(&F.flags[0], MST_FLAG_CORRUPT);
      }
      __syncthreads();
    }
    ++gpass;
  }
  const K tau = (K)sh.tau;
  const long long rem = sh.rem;
  const bool need_rank = sh.need_rank != 0;
  if (need_rank) {  // rank the entries equal to tau in index order
    if (CACHED) {
#pragma unroll
      for (int j = 0; j < KEYS_PER_LANE; ++j) {
        const int64_t w = lo + warp + (int64_t)j * FUSED_WARPS;
        if (w >= hi) break;
        const bool c = (candm >> j) & 1u;
        bool e = false;
        if (c) {
          if (MODE != MODE_RAND) e = (K)kc[j] == tau;
          else if ((K)kc[j] == (K)(tau >> (KB - 32))) e = cached_full_key(j) == tau;
        }
        const unsigned eq = __ballot_sync(0xffffffffu, e);
        if (lane == 0) F.cnt[w] = __popc(eq);
      }
    } else if (CACHE == CACHE_SMEM) {
      for (int64_t w = lo + warp; w < hi; w += FUSED_WARPS) {
        const uint32_t kw = skey[(w - lo) * 32 + lane];
        const bool c = (scand[w - lo] >> lane) & 1u;
        bool e = false;
        if (c) {
          if (MODE != MODE_RAND) e = (K)kw == tau;
          else if ((K)kw == (K)(tau >> (KB - 32))) e = word_full_key(w) == tau;
        }
        const unsigned eq = __ballot_sync(0xffffffffu, e);
        if (lane == 0) F.cnt[w] = __popc(eq);
      }
    } else
    for (int64_t w = lo + warp; w < hi; w += FUSED_WARPS) {
      unsigned long long key64;
      bool nf;
      const bool c = cand_key_w<MODE>(P, w, lane, s_old[w - lo], s_base[w - lo], s_grad[w - lo], key64, nf);
      const unsigned eq = __ballot_sync(0xffffffffu, c && (K)key64 == tau);
      if (lane == 0) F.cnt[w] = __popc(eq);
    }
    __syncthreads();
    fused_grid_scan(F.cnt, F.scan, P.nwords, lo, hi, F.bsums, gscan, grid, sh);
  }
  constexpr int MB = 4;
  if (CACHED) {
#pragma unroll
    for (int j = 0; j < KEYS_PER_LANE; ++j) {
      const int64_t w = lo + warp + (int64_t)j * FUSED_WARPS;
      if (w >= hi) break;  // uniform over the warp
      const bool c = (candm >> j) & 1u;
      bool below = false, equal = false;
      if (c) {
        if (MODE != MODE_RAND) {
          below = (K)kc[j] < tau;
          equal = (K)kc[j] == tau;
        } else {
          const K th = (K)(tau >> (KB - 32));
          if ((K)kc[j] < th) below = true;
          else if ((K)kc[j] == th) {
            const K key = cached_full_key(j);
            below = key < tau;
            equal = key == tau;
          }
        }
      }
      const unsigned eq = __ballot_sync(0xffffffffu, equal);
      const long long rank = need_rank ? (long long)F.scan[w] + __popc(eq & lanemask_lt()) : -1;
      const bool take = below || (equal && rank < rem);
      const unsigned bits = __ballot_sync(0xffffffffu, take);
      if (lane == 0) {
        out_bits[w] = bits;
        if (MODE == MODE_GRAD) s_grad[w - lo] = bits;
      }
    }
  } else if (CACHE == CACHE_SMEM) {
    for (int64_t w = lo + warp; w < hi; w += FUSED_WARPS) {
      const uint32_t kw = skey[(w - lo) * 32 + lane];
      const bool c = (scand[w - lo] >> lane) & 1u;
      bool below = false, equal = false;
      if (c) {
        if (MODE != MODE_RAND) {
          below = (K)kw < tau;
          equal = (K)kw == tau;
        } else {
          const K th = (K)(tau >> (KB - 32));
          if ((K)kw < th) below = true;
          else if ((K)kw == th) {
            const K key = word_full_key(w);
            below = key < tau;
            equal = key == tau;
          }
        }
      }
      const unsigned eq = __ballot_sync(0xffffffffu, equal);
      const long long rank = need_rank ? (long long)F.scan[w] + __popc(eq & lanemask_lt()) : -1;
      const bool take = below || (equal && rank < rem);
      const unsigned bits = __ballot_sync(0xffffffffu, take);
      if (lane == 0) {
        out_bits[w] = bits;
        if (MODE == MODE_GRAD) s_grad[w - lo] = bits;
      }
    }
  } else
  for (int64_t w0 = lo + warp; w0 < hi; w0 += FUSED_WARPS * MB) {
    bool c[MB], iseq[MB];
    K key[MB];
#pragma unroll
    for (int j = 0; j < MB; ++j) {
      const int64_t w = w0 + (int64_t)j * FUSED_WARPS;
      bool nf = false;
      unsigned long long key64 = 0;
      const int64_t li = w < hi ? w - lo : 0;
      c[j] = w < hi && cand_key_w<MODE>(P, w, lane, s_old[li], s_base[li], s_grad[li], key64, nf);
      key[j] = (K)key64;
      iseq[j] = c[j] && key[j] == tau;
    }
#pragma unroll
    for (int j = 0; j < MB; ++j) {
      const int64_t w = w0 + (int64_t)j * FUSED_WARPS;
      if (w >= hi) continue;  // uniform over the warp
      const unsigned eq = __ballot_sync(0xffffffffu, iseq[j]);
      const long long rank = need_rank ? (long long)F.scan[w] + __popc(eq & lanemask_lt()) : -1;
      const bool take = c[j] && (key[j] < tau || (iseq[j] && rank < rem));
      const unsigned bits = __ballot_sync(0xffffffffu, take);
      if (lane == 0) {
        out_bits[w] = bits;
        if (MODE == MODE_GRAD) s_grad[w - lo] = bits;  // the random selection of this block reads it from here
      }
    }
  }
  __syncthreads();
  UPD_STAMP(60 + MODE);
}

// ---------------------------------------------------------------------------------- two selections side by side
// Under the default reading of the candidate sets the prune selection looks only at active entries and the gradient
// selection only at inactive ones, so every entry carries exactly one 32-bit key and the two radix selects can share
// their sweeps and their barriers: pass p of both runs in one sweep into two histograms, both digits are picked behind
// one barrier, and one marking sweep writes both bit masks.

// columns of mask word w that exist (the last word of a row is ragged when I is not a multiple of 32)
__device__ __forceinline__ uint32_t word_valid_mask(const SelParams& P, int64_t w) {
  if (P.aligned) return 0xFFFFFFFFu;
  const unsigned wu = (unsigned)w, wpr = (unsigned)P.wpr;
  const int c0 = (int)(wu % wpr) * 32;
  const int nv = P.I - c0;
  return nv >= 32 ? 0xFFFFFFFFu : ((1u << nv) - 1u);
}

__device__ __forceinline__ long long word_flat_index(const SelParams& P, int64_t w, int lane) {
  if (P.aligned) return (long long)w * 32 + lane;
  const unsigned wu = (unsigned)w, wpr = (unsigned)P.wpr;
  const int o = (int)(wu / wpr), c = (int)(wu - (unsigned)o * wpr) * 32 + lane;
  return (long long)o * P.I + c;
}

// digit picks of the two selections from their complete histograms gh[0..BINS) and gh[BINS..2 BINS) (every block, same
// result); `todo` bit s: selection s still runs
__device__ void dual_pick(FusedShared& sh, unsigned todo, const unsigned int* gh, int shift, int width, int low_zero_a,
                          int32_t* flags) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned int mine[2][FUSED_BPT];
  unsigned int tsum[2] = {0u, 0u}, incl[2];
#pragma unroll
  for (int s = 0; s < 2; ++s) {
#pragma unroll
    for (int j = 0; j < FUSED_BPT; ++j) {
      mine[s][j] = ((todo >> s) & 1u) ? __ldcg(gh + s * BINS + threadIdx.x * FUSED_BPT + j) : 0u;
      tsum[s] += mine[s][j];
    }
  }
#pragma unroll
  for (int s = 0; s < 2; ++s) {
    incl[s] = tsum[s];
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned int y = __shfl_up_sync(0xffffffffu, incl[s], o);
      if (lane >= o) incl[s] += y;
    }
  }
  const uint32_t prefix[2] = {sh.d_prefix[0], sh.d_prefix[1]};
  const long long k[2] = {sh.d_k[0], sh.d_k[1]};
  __syncthreads();  // the totals' arrays are free, every thread has read the selection state
  if (threadIdx.x < 2) sh.d_found[threadIdx.x] = 0;
  if (lane == 31) {
    sh.warp_tot[warp] = incl[0];
    sh.red[warp] = (int)incl[1];
  }
  __syncthreads();
#pragma unroll
  for (int s = 0; s < 2; ++s) {
    if (!((todo >> s) & 1u)) continue;  // uniform
    unsigned int before = incl[s] - tsum[s];
    for (int wv = 0; wv < warp; ++wv) before += s ? (unsigned int)sh.red[wv] : sh.warp_tot[wv];
    const bool owner = (long long)before < k[s] && k[s] <= (long long)before + (long long)tsum[s];
    if (owner) {
      long long cum = before;
      int bin = 0;
      unsigned int bcount = 0;
      for (int j = 0; j < FUSED_BPT; ++j) {
        if (cum + (long long)mine[s][j] >= k[s]) { bin = j; bcount = mine[s][j]; break; }
        cum += mine[s][j];
      }
      const uint32_t np = (width < 32 ? (prefix[s] << width) : 0u) | (uint32_t)(threadIdx.x * FUSED_BPT + bin);
      sh.d_prefix[s] = np;
      sh.d_k[s] = k[s] - cum;
      sh.d_found[s] = 1;
      if (shift == 0) {
        sh.d_tau[s] = np;
        sh.d_rem[s] = k[s] - cum;
        sh.d_need_rank[s] = ((long long)bcount > k[s] - cum) ? 1 : 0;
        sh.d_done[s] = 1;
      } else if ((long long)bcount == k[s] - cum) {
        sh.d_tau[s] = (np << shift) | ((1u << shift) - 1u);
        sh.d_rem[s] = k[s] - cum;
        sh.d_need_rank[s] = 0;
        sh.d_done[s] = 1;
      } else if (s == 0 && shift <= low_zero_a) {
        // the undecided low bits are zero in every prune key: the bucket is one run of equal keys
        sh.d_tau[s] = np << shift;
        sh.d_rem[s] = k[s] - cum;
        sh.d_need_rank[s] = 1;
        sh.d_done[s] = 1;
      }
    }
  }
  __syncthreads();
  if (threadIdx.x < 2 && ((todo >> threadIdx.x) & 1u) && !sh.d_found[threadIdx.x]) {
    // fewer candidates than requested (ruled out by the host counts): take everything
    const int s = threadIdx.x;
    sh.d_tau[s] = 0xFFFFFFFFu;
    sh.d_rem[s] = 0x7FFFFFFFFFFFFFFFLL;
    sh.d_need_rank[s] = 0;
    sh.d_done[s] = 1;
    if (blockIdx.x == 0) atomicOr(&flags[0], MST_FLAG_CORRUPT);
  }
  __syncthreads();
}

// Shared-memory arrays of a block's slice in the side-by-side form of the update (one entry per mask word, keys one
// per entry).
struct DualSlice {
  uint32_t* old;   // mask words before the update
  int32_t* base;   // their exclusive popcount scan (position of a word's first entry in the value array)
  uint32_t* grad;  // entries grown by gradient
  uint32_t* prn;   // entries pruned
  uint32_t* hc;    // random growth: inactive entries whose hash can still be below the bracket's upper end
  uint32_t* key;   // [words][32] the 32-bit key of every entry
};

__device__ __forceinline__ unsigned long long entry_hash(const SelParams& P, long long f) {
  return sm64_mix(P.stream + SM64_GAMMA * ((unsigned long long)f + 1ULL));
}

// Prune and gradient selections side by side over keys kept in shared memory, random growth by bracket, mask rewrite.
// Sweeps over the slice: (0) keys, first histogram pass and the hash test of every inactive entry; (1, 2) the later
// histogram passes; (3) marking of pruned and gradient-grown entries, then one thread per word lists the random
// candidates inside the bracket; (4) behind the bracket's barrier, one thread per word marks the randomly grown
// entries and writes the new mask word.  Returns false (uniform over the grid) when the random growth still has to
// be done by the general radix select (no bracket, or the bracket missed); the new mask is not written then.
__device__ bool fused_dual_update(const FusedParams& F, int64_t lo, int nloc, int& gpass, int& gscan, cg::grid_group& grid,
                                  FusedShared& sh, const DualSlice& S) {
  const SelParams& P = F.sel;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const bool wantA = F.n_prune > 0, wantB = F.n_grad > 0;
  const bool wantR = F.rand_bracket && F.n_rand > 0;
  const bool aligned = P.aligned != 0;
  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      sh.d_prefix[s] = 0;
      sh.d_k[s] = s ? F.n_grad : F.n_prune;
      sh.d_tau[s] = 0;
      sh.d_rem[s] = 0;
      sh.d_need_rank[s] = 0;
      sh.d_done[s] = (s ? wantB : wantA) ? 0 : 1;
    }
  }
  for (int b = threadIdx.x; b < BINS; b += FUSED_THREADS) sh.hist[b] = 0;
  __syncthreads();
  // ---- sweep 0
  {
    const uint32_t rhi_hi = (uint32_t)(F.rand_hi >> 32);
    const bool lam = P.lambda != 0.f;
    bool saw_nonfinite = false;
    const bool bulk = F.g_bulk && wantB;   // uniform over the grid
    if (bulk) {
      // mask words tile the flat index space: the slice's gradients are one contiguous run, copied asynchronously
      // into the key array while the hashes below are computed
      const float* src = P.G + lo * 32;
      const uint32_t dst = (uint32_t)__cvta_generic_to_shared(S.key);
      for (int i = threadIdx.x; i < nloc * 8; i += FUSED_THREADS)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 16u * (uint32_t)i), "l"(src + 4 * (size_t)i) : "memory");
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    // random growth: which inactive entries have a hash whose high word does not exceed the bracket's upper end
    if (wantR && aligned) {
      // flat index (lo + li) * 32 + lane: the generator's argument advances by a constant from one of this warp's
      // words to the next
      unsigned long long z = P.stream + SM64_GAMMA * ((unsigned long long)(lo + warp) * 32ULL + (unsigned long long)lane + 1ULL);
      constexpr unsigned long long ZSTEP = SM64_GAMMA * 32ULL * (unsigned long long)FUSED_WARPS;
#pragma unroll 4
      for (int li = warp; li < nloc; li += FUSED_WARPS) {
        const bool act = (S.old[li] >> lane) & 1u;
        const bool h_ok = !act && (uint32_t)(sm64_mix(z) >> 32) <= rhi_hi;
        z += ZSTEP;
        const unsigned hm = __ballot_sync(0xffffffffu, h_ok);
        if (lane == 0) S.hc[li] = hm;
      }
    } else if (wantR) {
#pragma unroll 4
      for (int li = warp; li < nloc; li += FUSED_WARPS) {
        const bool act = (S.old[li] >> lane) & 1u;
        const bool valid = (word_valid_mask(P, lo + li) >> lane) & 1u;
        bool h_ok = false;
        if (!act && valid) h_ok = (uint32_t)(entry_hash(P, word_flat_index(P, lo + li, lane)) >> 32) <= rhi_hi;
        const unsigned hm = __ballot_sync(0xffffffffu, h_ok);
        if (lane == 0) S.hc[li] = hm;
      }
    } else {
      for (int li = threadIdx.x; li < nloc; li += FUSED_THREADS) S.hc[li] = 0u;
    }
    UPD_STAMP(4);
    if (bulk) {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncthreads();
    }
    // gradient keys of the inactive entries, lane per entry (the active entries' slots are written below)
    if (wantB) {
      constexpr int GB = 4;  // words per trip, loads first
      for (int l0 = warp; l0 < nloc; l0 += FUSED_WARPS * GB) {
        uint32_t kk[GB], ow[GB];
#pragma unroll
        for (int j = 0; j < GB; ++j) {
          const int li = l0 + j * FUSED_WARPS;
          kk[j] = 0u;
          ow[j] = 0xFFFFFFFFu;
          if (li < nloc) {  // uniform over the warp
            ow[j] = S.old[li];
            const bool c = !((ow[j] >> lane) & 1u) && (aligned || ((word_valid_mask(P, lo + li) >> lane) & 1u));
            if (bulk) kk[j] = S.key[li * 32 + lane] & 0x7FFFFFFFu;
            else if (c) kk[j] = __float_as_uint(P.G[word_flat_index(P, lo + li, lane)]) & 0x7FFFFFFFu;
          }
        }
#pragma unroll
        for (int j = 0; j < GB; ++j) {
          const int li = l0 + j * FUSED_WARPS;
          if (li >= nloc) break;  // uniform over the warp
          const bool c = !((ow[j] >> lane) & 1u) && (aligned || ((word_valid_mask(P, lo + li) >> lane) & 1u));
          const uint32_t key = 0xFFFFFFFFu - kk[j];  // largest magnitude first
          if (c) {
            saw_nonfinite |= kk[j] >= 0x7F800000u;
            atomicAdd(&sh.hist[key >> pass_shift(32, 0)], 0x10000u);
          }
          S.key[li * 32 + lane] = key;
        }
      }
      __syncthreads();  // the active entries' slots are rewritten by other threads below
    }
    // prune keys of the active entries, one thread per word
    if (wantA) {
      for (int li = threadIdx.x; li < nloc; li += FUSED_THREADS) {
        uint32_t m = S.old[li];
        int32_t pos = S.base[li];
        while (m) {
          const int b = __ffs(m) - 1;
          m &= m - 1;
          uint32_t k = (P.bf16 ? (uint32_t)((const uint16_t*)P.vals)[pos] << 16 : ((const uint32_t*)P.vals)[pos]) & 0x7FFFFFFFu;
          ++pos;
          if (lam) {  // MEST criterion, fp32 with one rounding per operation (never contracted to an FMA)
            const float g = fabsf(P.G[word_flat_index(P, lo + li, b)]);
            k = __float_as_uint(__fadd_rn(__uint_as_float(k), __fmul_rn(P.lambda, g))) & 0x7FFFFFFFu;
          }
          saw_nonfinite |= k >= 0x7F800000u;
          S.key[li * 32 + b] = k;
          atomicAdd(&sh.hist[k >> pass_shift(32, 0)], 1u);
        }
      }
    }
    if (saw_nonfinite) atomicOr(&F.flags[0], MST_FLAG_NONFINITE);
  }
  UPD_STAMP(3);
  // ---- histogram passes (the first one was filled by sweep 0)
  constexpr int passes = num_passes(32);
  for (int pass = 0; pass < passes; ++pass) {
    const bool doneA = sh.d_done[0] != 0, doneB = sh.d_done[1] != 0;
    if (doneA && doneB) break;  // same decision in every block
    const int shift = pass_shift(32, pass), width = pass_width(32, pass);
    unsigned int* gh = F.hist + (gpass % 3) * HSTRIDE;
    if (pass > 0) {
      const unsigned dmask = (1u << width) - 1u;
      const int hi_shift = shift + width;
      const uint32_t prefA = sh.d_prefix[0], prefB = sh.d_prefix[1];
      const bool liveA = wantA && !doneA, liveB = wantB && !doneB;
      __syncthreads();  // every thread has read the selection state
      for (int b = threadIdx.x; b < BINS; b += FUSED_THREADS) sh.hist[b] = 0;
      __syncthreads();
      constexpr int PB = 4;  // words per trip: the shared-memory atomics would otherwise keep the next loads behind them
      for (int l0 = warp; l0 < nloc; l0 += FUSED_WARPS * PB) {
        uint32_t key[PB], ow[PB];
#pragma unroll
        for (int j = 0; j < PB; ++j) {
          const int li = l0 + j * FUSED_WARPS;
          const bool ok = li < nloc;  // uniform over the warp
          key[j] = ok ? S.key[li * 32 + lane] : 0u;
          ow[j] = ok ? S.old[li] : 0u;
        }
#pragma unroll
        for (int j = 0; j < PB; ++j) {
          const int li = l0 + j * FUSED_WARPS;
          if (li >= nloc) break;  // uniform over the warp
          const bool act = (ow[j] >> lane) & 1u;
          const bool valid = aligned || ((word_valid_mask(P, lo + li) >> lane) & 1u);
          const bool lv = (act ? liveA : (liveB && valid)) && (key[j] >> hi_shift) == (act ? prefA : prefB);
          if (lv) atomicAdd(&sh.hist[(key[j] >> shift) & dmask], act ? 1u : 0x10000u);
        }
      }
    }
    __syncthreads();
    UPD_STAMP(10 + pass);
    for (int b = threadIdx.x; b < BINS; b += FUSED_THREADS) {
      const unsigned int v = sh.hist[b];
      if (v & 0xFFFFu) atomicAdd(&gh[b], v & 0xFFFFu);
      if (v >> 16) atomicAdd(&gh[BINS + b], v >> 16);
    }
    grid.sync();
    UPD_STAMP(20 + pass);
    dual_pick(sh, (doneA ? 0u : 1u) | (doneB ? 0u : 2u), gh, shift, width, P.low_zero, F.flags);
    if (blockIdx.x == 0) {  // clear the buffer of pass gpass + 2 (last read before this barrier)
      unsigned int* gz = F.hist + ((gpass + 2) % 3) * HSTRIDE;
      for (int b = threadIdx.x; b < HSTRIDE; b += FUSED_THREADS) gz[b] = 0;
    }
    __syncthreads();
    UPD_STAMP(30 + pass);
    ++gpass;
  }
  const uint32_t tauA = sh.d_tau[0], tauB = sh.d_tau[1];
  const long long remA = sh.d_rem[0], remB = sh.d_rem[1];
  const bool rankA = sh.d_need_rank[0] != 0, rankB = sh.d_need_rank[1] != 0;
  // tie ranking in index order, one scan per selection that needs it (the second into the array of the new mask's
  // scan, which is not written before the mask rewrite)
  for (int s = 0; s < 2; ++s) {
    if (!(s ? rankB : rankA)) continue;  // uniform over the grid
    const uint32_t tau = s ? tauB : tauA;
    for (int li = warp; li < nloc; li += FUSED_WARPS) {
      const bool act = (S.old[li] >> lane) & 1u;
      const bool valid = aligned || ((word_valid_mask(P, lo + li) >> lane) & 1u);
      const bool c = s ? (!act && valid) : act;
      const unsigned eq = __ballot_sync(0xffffffffu, c && S.key[li * 32 + lane] == tau);
      if (lane == 0) F.cnt[lo + li] = __popc(eq);
    }
    __syncthreads();
    fused_grid_scan(F.cnt, s ? F.new_wscan : F.scan, P.nwords, lo, lo + nloc, F.bsums, gscan, grid, sh);
  }
  UPD_STAMP(40);
  // ---- sweep 3: marking
  if (!rankA && !rankB) {
    // no tie has to be ranked: an entry is taken when its key does not exceed its selection's threshold
    const uint32_t enA = wantA ? 0xFFFFFFFFu : 0u, enB = wantB ? 0xFFFFFFFFu : 0u;
    constexpr int MB = 4;  // words per trip, loads first
    for (int l0 = warp; l0 < nloc; l0 += FUSED_WARPS * MB) {
      uint32_t key[MB], ow[MB];
#pragma unroll
      for (int j = 0; j < MB; ++j) {
        const int li = l0 + j * FUSED_WARPS;
        const bool ok = li < nloc;  // uniform over the warp
        key[j] = ok ? S.key[li * 32 + lane] : 0u;
        ow[j] = ok ? S.old[li] : 0u;
      }
#pragma unroll
      for (int j = 0; j < MB; ++j) {
        const int li = l0 + j * FUSED_WARPS;
        if (li >= nloc) break;  // uniform over the warp
        const bool act = (ow[j] >> lane) & 1u;
        const unsigned all = __ballot_sync(0xffffffffu, key[j] <= (act ? tauA : tauB));
        if (lane == 0) {
          S.prn[li] = all & ow[j] & enA;
          S.grad[li] = all & ~ow[j] & enB & (aligned ? 0xFFFFFFFFu : word_valid_mask(P, lo + li));
        }
      }
    }
  } else
  for (int li = warp; li < nloc; li += FUSED_WARPS) {
    const uint32_t key = S.key[li * 32 + lane];
    const bool act = (S.old[li] >> lane) & 1u;
    const bool valid = aligned || ((word_valid_mask(P, lo + li) >> lane) & 1u);
    bool takeA = wantA && act && key < tauA, takeB = wantB && !act && valid && key < tauB;
    const bool eqA = wantA && act && key == tauA, eqB = wantB && !act && valid && key == tauB;
    if (rankA) {  // uniform
      const unsigned m = __ballot_sync(0xffffffffu, eqA);
      takeA |= eqA && (long long)F.scan[lo + li] + __popc(m & lanemask_lt()) < remA;
    } else {
      takeA |= eqA;
    }
    if (rankB) {
      const unsigned m = __ballot_sync(0xffffffffu, eqB);
      takeB |= eqB && (long long)F.new_wscan[lo + li] + __popc(m & lanemask_lt()) < remB;
    } else {
      takeB |= eqB;
    }
    const unsigned bA = __ballot_sync(0xffffffffu, takeA), bB = __ballot_sync(0xffffffffu, takeB);
    if (lane == 0) {
      S.prn[li] = bA;
      S.grad[li] = bB;
    }
  }
  __syncthreads();
  UPD_STAMP(41);
  if (!wantR && F.n_rand > 0) return false;  // uniform over the grid: no bracket was planned
  if (wantR) {
    // one thread per word: the remaining candidates whose hash lies below the bracket are counted, those inside
    // listed (counted first, so that a block reserves its part of the list with one atomic)
    unsigned long long below_lo = 0;
    int n_in = 0;
    for (int li = threadIdx.x; li < nloc; li += FUSED_THREADS) {
      uint32_t m = S.hc[li] & ~S.grad[li], keep = 0;
      while (m) {
        const int b = __ffs(m) - 1;
        m &= m - 1;
        const unsigned long long h = entry_hash(P, word_flat_index(P, lo + li, b));
        if (h < F.rand_lo) {
          ++below_lo;
          keep |= 1u << b;
        } else if (h < F.rand_hi) {
          ++n_in;
          keep |= 1u << b;
        }
      }
      S.hc[li] = keep;  // what can still be taken
    }
    int blk_in = 0;
    const int my_at = fused_block_excl_scan(n_in, blk_in, sh);
    __syncthreads();
    if (threadIdx.x == 0) sh.r_tau = blk_in ? atomicAdd(&F.rand_ctr[1], (unsigned long long)blk_in) : 0ULL;
    __syncthreads();
    if (n_in) {
      unsigned long long at = sh.r_tau + (unsigned long long)my_at;
      for (int li = threadIdx.x; li < nloc; li += FUSED_THREADS) {
        uint32_t m = S.hc[li];
        while (m) {
          const int b = __ffs(m) - 1;
          m &= m - 1;
          const long long f = word_flat_index(P, lo + li, b);
          const unsigned long long h = entry_hash(P, f);
          if (h >= F.rand_lo) {
            if (at < (unsigned long long)F.rand_cap) {
              F.rand_list[2 * at] = h;
              F.rand_list[2 * at + 1] = (unsigned long long)f;
            }
            ++at;
          }
        }
      }
    }
    for (int o = 16; o; o >>= 1) below_lo += __shfl_xor_sync(0xffffffffu, below_lo, o);
    if (lane == 0 && below_lo) atomicAdd(&F.rand_ctr[0], below_lo);
    grid.sync();
    UPD_STAMP(42);
    const unsigned long long c_lo = __ldcg(&F.rand_ctr[0]), n_list = __ldcg(&F.rand_ctr[1]);
    const unsigned long long k = (unsigned long long)F.n_rand;
    if (!(c_lo < k && k <= c_lo + n_list && n_list <= (unsigned long long)F.rand_cap)) return false;  // uniform over the grid
    const int n = (int)n_list;
    const long long r = (long long)(k - c_lo);  // 1-based rank inside the list
    const unsigned long long range = F.rand_hi - F.rand_lo;
    // bin of a key: (key - lo) >> bshift, below BINS because range >> bshift < BINS
    const int bshift = (range >> RADIX_BITS) ? 64 - RADIX_BITS - __clzll((long long)range) : 0;
    __syncthreads();
    for (int b = threadIdx.x; b < BINS; b += FUSED_THREADS) sh.hist[b] = 0;
    if (threadIdx.x == 0) { sh.r_ok = 0; sh.r_n = 0; }
    __syncthreads();
    // the keys of the selections are not needed any more: their array stages the listed hash keys
    unsigned long long* staged = reinterpret_cast<unsigned long long*>(S.key);
    const bool stage = n <= nloc * 16;  // uniform over the block
    for (int i = threadIdx.x; i < n; i += FUSED_THREADS) {
      const unsigned long long key = __ldcg(&F.rand_list[2 * (size_t)i]);
      if (stage) staged[i] = key;
      atomicAdd(&sh.hist[(unsigned)((key - F.rand_lo) >> bshift)], 1u);
    }
    __syncthreads();
    {
      unsigned int mine[FUSED_BPT];
      unsigned int tsum = 0;
#pragma unroll
      for (int j = 0; j < FUSED_BPT; ++j) {
        mine[j] = sh.hist[threadIdx.x * FUSED_BPT + j];
        tsum += mine[j];
      }
      unsigned int incl = tsum;
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
      }
      if (lane == 31) sh.warp_tot[warp] = incl;
      __syncthreads();
      unsigned int before = incl - tsum;
      for (int wv = 0; wv < warp; ++wv) before += sh.warp_tot[wv];
      if ((long long)before < r && r <= (long long)before + (long long)tsum) {
        long long cum = before;
        for (int j = 0; j < FUSED_BPT; ++j) {
          if (cum + (long long)mine[j] >= r) {
            sh.r_bin = threadIdx.x * FUSED_BPT + j;
            sh.r_rank = r - cum;                                  // 1-based rank inside the bin
            sh.r_ok = mine[j] <= (unsigned)(BINS / 4) ? 1 : 0;   // the bin's entries must fit the shared array below
            break;
          }
          cum += mine[j];
        }
      }
      __syncthreads();
    }
    if (!sh.r_ok) return false;  // same data in every block: same decision
    const unsigned rbin = (unsigned)sh.r_bin;
    const long long rr = sh.r_rank;
    __syncthreads();
    // the entries of that bin, gathered over the histogram's storage (BINS words = BINS / 4 pairs of 64-bit words)
    unsigned long long* small = reinterpret_cast<unsigned long long*>(sh.hist);
    for (int i = threadIdx.x; i < n; i += FUSED_THREADS) {
      const unsigned long long key = stage ? staged[i] : __ldcg(&F.rand_list[2 * (size_t)i]);
      if ((unsigned)((key - F.rand_lo) >> bshift) == rbin) {
        const int at = atomicAdd(&sh.r_n, 1);
        small[2 * at] = key;
        small[2 * at + 1] = __ldcg(&F.rand_list[2 * (size_t)i + 1]);
      }
    }
    __syncthreads();
    const int m = sh.r_n;
    for (int i = threadIdx.x; i < m; i += FUSED_THREADS) {
      const unsigned long long key = small[2 * i], f = small[2 * i + 1];
      int rank = 0;
      for (int q = 0; q < m; ++q) {
        const unsigned long long kq = small[2 * q], fq = small[2 * q + 1];
        rank += (kq < key || (kq == key && fq < f)) ? 1 : 0;
      }
      if (rank == (int)(rr - 1)) { sh.r_tau = key; sh.r_tau_f = f; }
    }
    __syncthreads();
    UPD_STAMP(43);
  }
  // ---- sweep 4, one thread per word: randomly grown entries and the new mask word
  const unsigned long long tau = wantR ? sh.r_tau : 0ULL, tau_f = wantR ? sh.r_tau_f : 0ULL;
  for (int li = threadIdx.x; li < nloc; li += FUSED_THREADS) {
    uint32_t m = wantR ? S.hc[li] : 0u, bR = 0;
    while (m) {
      const int b = __ffs(m) - 1;
      m &= m - 1;
      const unsigned long long f = (unsigned long long)word_flat_index(P, lo + li, b);
      const unsigned long long h = entry_hash(P, (long long)f);
      if (h < tau || (h == tau && f <= tau_f)) bR |= 1u << b;
    }
    const uint32_t nb = (S.old[li] & ~S.prn[li]) | S.grad[li] | bR;
    F.new_bits[lo + li] = nb;
    F.cnt[lo + li] = __popc(nb);
    S.hc[li] = nb;  // for the rebuild below
  }
  __syncthreads();
  UPD_STAMP(44);
  return true;
}

// Scan of the new mask and CSR fill from the slice kept in shared memory (new mask words in S.hc): the same result
// as fused_grid_scan + mst_fill_csr_words, without fetching masks and scans again.  One grid barrier inside.
template <typename V>
__device__ void fused_dual_rebuild(const FusedParams& F, int64_t lo, int nloc, int& gscan, cg::grid_group& grid,
                                   FusedShared& sh, const DualSlice& S) {
  const SelParams& P = F.sel;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int32_t* bsums = F.bsums + (gscan & 1) * (int)gridDim.x;
  ++gscan;
  int v = 0;
  for (int li = threadIdx.x; li < nloc; li += FUSED_THREADS) v += __popc(S.hc[li]);
  const int bs = fused_block_sum(v, sh);
  if (threadIdx.x == 0) bsums[blockIdx.x] = bs;
  grid.sync();
  int off = 0, tot = 0;
  for (int j = threadIdx.x; j < (int)gridDim.x; j += FUSED_THREADS) {
    const int x = __ldcg(bsums + j);
    tot += x;
    if (j < (int)blockIdx.x) off += x;
  }
  off = fused_block_sum(off, sh);
  tot = fused_block_sum(tot, sh);
  int carry = off;
  int32_t* nbase = reinterpret_cast<int32_t*>(S.prn);  // the pruned bits are not needed any more
  for (int b0 = 0; b0 < nloc; b0 += FUSED_THREADS) {
    const int li = b0 + threadIdx.x;
    const int x = li < nloc ? __popc(S.hc[li]) : 0;
    int tile_total;
    const int ex = fused_block_excl_scan(x, tile_total, sh);
    if (li < nloc) {
      nbase[li] = carry + ex;
      F.new_wscan[lo + li] = carry + ex;
    }
    carry += tile_total;
  }
  if (threadIdx.x == 0) F.new_wscan[P.nwords] = tot;
  __syncthreads();
  UPD_STAMP(52);
  // fill, one thread per word: a word holds few entries, and the lanes of a warp-per-word loop would mostly idle
  const V* old_vals = (const V*)P.vals;
  V* new_vals = (V*)F.new_vals;
  for (int li = threadIdx.x; li < nloc; li += FUSED_THREADS) {
    const uint32_t nb = S.hc[li], ob = S.old[li];
    const unsigned wu = (unsigned)(lo + li);
    const int o = (int)(wu / (unsigned)P.wpr), wc = (int)(wu - (unsigned)o * (unsigned)P.wpr);
    int32_t pos = nbase[li];
    if (wc == 0) {
      F.new_row_ptr[o] = pos;
      if (o == P.O - 1) F.new_row_ptr[P.O] = tot;
    }
    const int32_t obase = S.base[li];
    uint32_t m = nb;
    while (m) {
      const int b = __ffs(m) - 1;
      m &= m - 1;
      V v = V(0);
      if ((ob >> b) & 1u) v = old_vals[obase + __popc(ob & ((1u << b) - 1u))];
      F.new_col[pos] = (uint16_t)(wc * 32 + b);
      new_vals[pos] = v;
      ++pos;
    }
  }
}

template <typename V>
__global__ void __launch_bounds__(FUSED_THREADS, 2) mg_update_fused_kernel(const FusedParams F) {
  cg::grid_group grid = cg::this_grid();
  __shared__ FusedShared sh;
  mst_grid_launch_dependents();
  mst_grid_dependency_wait();
  const SelParams& P = F.sel;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t per = (P.nwords + gridDim.x - 1) / gridDim.x;
  const int64_t lo = per * blockIdx.x < P.nwords ? per * blockIdx.x : P.nwords;
  const int64_t hi = lo + per < P.nwords ? lo + per : P.nwords;
  const int64_t perT = (F.nwordsT + gridDim.x - 1) / gridDim.x;
  const int64_t loT = perT * blockIdx.x < F.nwordsT ? perT * blockIdx.x : F.nwordsT;
  const int64_t hiT = loT + perT < F.nwordsT ? loT + perT : F.nwordsT;

  // this block's slice of the old mask and of its scan stays in shared memory for every selection pass
  extern __shared__ __align__(16) uint32_t s_dyn[];
  uint32_t* skey = s_dyn;                     // only present (and used) when the launch asked for the key cache
  uint32_t* s_small = s_dyn + (F.smem_keys ? 32 * per : 0);
  uint32_t* s_old = s_small;
  int32_t* s_base = reinterpret_cast<int32_t*>(s_small + per);
  uint32_t* s_grad = s_small + 2 * per;
  uint32_t* scand = s_small + 3 * per;        // candidate words of the running selection
  uint32_t* s_prn = s_small + 4 * per;        // side-by-side form: pruned bits
  for (int64_t w = lo + threadIdx.x; w < hi; w += FUSED_THREADS) {
    s_old[w - lo] = P.old_bits[w];
    s_base[w - lo] = P.old_wscan[w];
    s_grad[w - lo] = 0;
  }
  if (blockIdx.x == 0 && threadIdx.x < 3) F.flags[1 + threadIdx.x] = 0;  // per-update statistics (first used behind a barrier)
#ifdef MST_UPD_PROFILE
  if (blockIdx.x == 0 && threadIdx.x == 0) g_upd_nstamps = 0;
#endif
  __syncthreads();
  UPD_STAMP(2);

  int gpass = 0, gscan = 0;
  const int cache = F.smem_keys ? CACHE_SMEM : (per <= (int64_t)FUSED_WARPS * KEYS_PER_LANE ? CACHE_REGS : CACHE_NONE);  // uniform over the grid
  bool rewritten = false;
  if (F.dual) {  // the launch carries the key cache
    DualSlice S;
    S.old = s_old; S.base = s_base; S.grad = s_grad; S.prn = s_prn; S.hc = scand; S.key = skey;
    rewritten = fused_dual_update(F, lo, (int)(hi - lo), gpass, gscan, grid, sh, S);
  } else if (cache == CACHE_REGS) {
    fused_select<MODE_PRUNE, CACHE_REGS>(F, F.n_prune, F.pruned_bits, lo, hi, gpass, gscan, grid, sh, s_old, s_base, s_grad, skey, scand);
    fused_select<MODE_GRAD, CACHE_REGS>(F, F.n_grad, F.grad_bits, lo, hi, gpass, gscan, grid, sh, s_old, s_base, s_grad, skey, scand);
  } else if (cache == CACHE_SMEM) {
    fused_select<MODE_PRUNE, CACHE_SMEM>(F, F.n_prune, F.pruned_bits, lo, hi, gpass, gscan, grid, sh, s_old, s_base, s_grad, skey, scand);
    fused_select<MODE_GRAD, CACHE_SMEM>(F, F.n_grad, F.grad_bits, lo, hi, gpass, gscan, grid, sh, s_old, s_base, s_grad, skey, scand);
  } else {
    fused_select<MODE_PRUNE, CACHE_NONE>(F, F.n_prune, F.pruned_bits, lo, hi, gpass, gscan, grid, sh, s_old, s_base, s_grad, skey, scand);
    fused_select<MODE_GRAD, CACHE_NONE>(F, F.n_grad, F.grad_bits, lo, hi, gpass, gscan, grid, sh, s_old, s_base, s_grad, skey, scand);
  }
  UPD_STAMP(49);
  if (!rewritten) {  // uniform over the grid: random growth by the general radix select, then the mask rewrite
    if (cache == CACHE_REGS)
      fused_select<MODE_RAND, CACHE_REGS>(F, F.n_rand, F.rand_bits, lo, hi, gpass, gscan, grid, sh, s_old, s_base, s_grad, skey, scand);
    else if (cache == CACHE_SMEM)
      fused_select<MODE_RAND, CACHE_SMEM>(F, F.n_rand, F.rand_bits, lo, hi, gpass, gscan, grid, sh, s_old, s_base, s_grad, skey, scand);
    else
      fused_select<MODE_RAND, CACHE_NONE>(F, F.n_rand, F.rand_bits, lo, hi, gpass, gscan, grid, sh, s_old, s_base, s_grad, skey, scand);
    // mask rewrite: new = (old & ~pruned) | grad | rand, and its popcounts
    for (int64_t w = lo + threadIdx.x; w < hi; w += FUSED_THREADS) {
      const uint32_t pw = F.dual ? s_prn[w - lo] : F.pruned_bits[w], gw = F.dual ? s_grad[w - lo] : F.grad_bits[w];
      const uint32_t b = (s_old[w - lo] & ~pw) | gw | F.rand_bits[w];
      F.new_bits[w] = b;
      F.cnt[w] = __popc(b);
    }
    __syncthreads();
  }
  UPD_STAMP(51);
  if (rewritten && !F.build_csc) {  // uniform over the grid: the slice's new mask is still in shared memory
    DualSlice S;
    S.old = s_old; S.base = s_base; S.grad = s_grad; S.prn = s_prn; S.hc = scand; S.key = skey;
    fused_dual_rebuild<V>(F, lo, (int)(hi - lo), gscan, grid, sh, S);
    UPD_STAMP(53);
    if (blockIdx.x == 0) {  // every pick and every list read lies before the last barrier: leave the scratch zero
      for (int b = threadIdx.x; b < 3 * HSTRIDE; b += FUSED_THREADS) F.hist[b] = 0;
      if (threadIdx.x < 2) F.rand_ctr[threadIdx.x] = 0;
    }
    UPD_STAMP(54);
    return;
  }
  fused_grid_scan(F.cnt, F.new_wscan, P.nwords, lo, hi, F.bsums, gscan, grid, sh);
  UPD_STAMP(52);
  // the barrier inside the scan came after every block wrote its part of the new mask: transpose it now
  if (F.build_csc) {
    const int64_t tiles = (int64_t)F.wpc * P.wpr;
    for (int64_t t = (int64_t)blockIdx.x * FUSED_WARPS + warp; t < tiles; t += (int64_t)gridDim.x * FUSED_WARPS)
      mst_transpose_tile(t, lane, F.new_bits, P.O, P.I, P.wpr, F.wpc, F.bitsT);
    grid.sync();  // the transposed mask is complete everywhere
  }
  for (int64_t w0 = lo + warp; w0 < hi; w0 += FUSED_WARPS * 4)
    mst_fill_csr_words<V, 4>(w0, FUSED_WARPS, hi, lane, F.new_bits, F.new_wscan, P.O, P.wpr, F.new_col, (V*)F.new_vals,
                             F.new_row_ptr, P.old_bits, P.old_wscan, (const V*)P.vals,
                             F.build_csc ? &F.flags[1] : nullptr);  // without the barrier above the next row's scan entry
                                                                    // may belong to a block that has not written it yet
  UPD_STAMP(53);
  if (blockIdx.x == 0) {  // every pick and every list read lies before the last barrier: leave the scratch zero
    for (int b = threadIdx.x; b < 3 * HSTRIDE; b += FUSED_THREADS) F.hist[b] = 0;
    if (threadIdx.x < 2) F.rand_ctr[threadIdx.x] = 0;
  }
  UPD_STAMP(54);
  if (!F.build_csc) return;  // uniform over the grid
  for (int64_t w = loT + threadIdx.x; w < hiT; w += FUSED_THREADS) F.cnt[w] = __popc(F.bitsT[w]);
  __syncthreads();
  const int totT = fused_grid_scan(F.cnt, F.wscanT, F.nwordsT, loT, hiT, F.bsums, gscan, grid, sh);
  for (int64_t w0 = loT + warp; w0 < hiT; w0 += FUSED_WARPS * 4)
    mst_fill_csc_words<4>(w0, FUSED_WARPS, hiT, lane, F.bitsT, F.wscanT, P.I, P.wpr, F.wpc, F.new_bits, F.new_wscan,
                          F.row_idx, F.perm, F.col_ptr, totT);
}

// ------------------------------------------------------------------------------------------------ batched update
// The updates of several layers in ONE cooperative launch.  The single-layer kernel above is a chain of about ten
// grid-wide barriers with little work between them; here every round does, for each layer in turn, the work of that
// layer's current phase, and then ALL layers share one barrier.  A layer's phases and their order are those of the
// single-layer kernel (histogram pass -> digit pick, tie count -> scan -> mark, mask rewrite -> scan -> CSR fill), its
// selection state lives in shared memory per layer, and every block takes every decision from the same global
// histograms, so all blocks walk through the same sequence.  Results are bit-identical to updating the layers one
// after the other.  Keys are recomputed from global memory in every pass (no register cache: a block holds slices of
// all layers), and the CSC view is not built (layers that need it take the single-layer path).
constexpr int BATCH_MAX = 8;
enum { PH_NEW = 0, PH_HIST = 1, PH_TIE = 2, PH_REWRITE = 3, PH_DONE = 4 };

struct BatchParams {
  FusedParams L[BATCH_MAX];
  int smem_off[BATCH_MAX];  // word offset of the layer's three slices (old mask, its scan, gradient marks) in dynamic smem
  int n;
};

struct BatchLayerState {
  unsigned long long prefix, tau;
  long long k, rem;
  int need_rank, done, found;
  int sel;    // 0 prune, 1 gradient, 2 random, 3 rewrite
  int phase;  // which barrier the layer waits for next
  int pass, gpass, gscan;
};

struct BatchShared {
  unsigned int hist[BINS];
  unsigned int warp_tot[FUSED_WARPS];
  int red[FUSED_WARPS];
  BatchLayerState st[BATCH_MAX];
};

struct BatchSlice {
  int64_t lo, hi;
  uint32_t* s_old;
  int32_t* s_base;
  uint32_t* s_grad;
};

__device__ __forceinline__ int batch_block_sum(int v, int* red) {
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  int r = 0;
#pragma unroll
  for (int w = 0; w < FUSED_WARPS; ++w) r += red[w];
  return r;
}
__device__ __forceinline__ int batch_block_excl_scan(int v, int& total, int* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int x = v;
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  __syncthreads();
  if (lane == 31) red[warp] = x;
  __syncthreads();
  int before = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < FUSED_WARPS; ++w) {
    const int t = red[w];
    if (w < warp) before += t;
    tot += t;
  }
  total = tot;
  return before + x - v;
}

// first half of a grid-wide scan: this block's sum of cnt[lo, hi) into the layer's current partial-sum area
__device__ void batch_scan_begin(const int32_t* cnt, int64_t lo, int64_t hi, int32_t* bsums, int gscan, int* red) {
  int v = 0;
  for (int64_t i = lo + threadIdx.x; i < hi; i += FUSED_THREADS) v += cnt[i];
  const int bs = batch_block_sum(v, red);
  if (threadIdx.x == 0) bsums[(gscan & 1) * (int)gridDim.x + blockIdx.x] = bs;
}
// second half, behind the barrier: out[lo, hi) = exclusive scan, out[n] = total
__device__ int batch_scan_end(const int32_t* cnt, int32_t* out, int64_t n, int64_t lo, int64_t hi, const int32_t* bsums,
                               int gscan, int* red) {
  const int32_t* area = bsums + (gscan & 1) * (int)gridDim.x;
  int off = 0, tot = 0;
  for (int j = threadIdx.x; j < (int)gridDim.x; j += FUSED_THREADS) {
    const int x = __ldcg(area + j);
    tot += x;
    if (j < (int)blockIdx.x) off += x;
  }
  off = batch_block_sum(off, red);
  tot = batch_block_sum(tot, red);
  int carry = off;
  for (int64_t base = lo; base < hi; base += FUSED_THREADS) {
    const int64_t i = base + threadIdx.x;
    const int x = i < hi ? cnt[i] : 0;
    int tile_total;
    const int ex = batch_block_excl_scan(x, tile_total, red);
    if (i < hi) out[i] = carry + ex;
    carry += tile_total;
  }
  if (threadIdx.x == 0) out[n] = tot;
  __syncthreads();
  return tot;
}

template <int MODE>
__device__ void batch_hist_sweep(const FusedParams& F, BatchLayerState& st, const BatchSlice& sl, BatchShared& sh) {
  constexpr int KB = KeyBits<MODE>::value;
  typedef typename KeyWord<MODE>::type K;
  const SelParams& P = F.sel;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int pass = st.pass;
  const int shift = pass_shift(KB, pass), width = pass_width(KB, pass);
  const unsigned dmask = (1u << width) - 1u;
  const int hi_shift = shift + width;
  const K prefix = (K)st.prefix;
  unsigned int* gh = F.hist + (st.gpass % 3) * BINS;
  __syncthreads();  // the state was written by the previous step
  for (int b = threadIdx.x; b < BINS; b += FUSED_THREADS) sh.hist[b] = 0;
  __syncthreads();
  bool saw_nonfinite = false;
  constexpr int BATCH = 8;
  for (int64_t w0 = sl.lo + warp; w0 < sl.hi; w0 += FUSED_WARPS * BATCH) {
    unsigned digit[BATCH];
    bool live[BATCH];
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      const int64_t w = w0 + (int64_t)j * FUSED_WARPS;
      unsigned long long key64 = 0;
      bool nf = false;
      const int64_t li = w < sl.hi ? w - sl.lo : 0;
      const bool c = w < sl.hi && cand_key_w<MODE>(P, w, lane, sl.s_old[li], sl.s_base[li], sl.s_grad[li], key64, nf);
      const K key = (K)key64;
      saw_nonfinite |= (c && nf);
      live[j] = c && (pass == 0 || (K)(key >> hi_shift) == prefix);
      digit[j] = live[j] ? (unsigned)((key >> shift) & (K)dmask) : (unsigned)BINS;
    }
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      if (live[j]) atomicAdd(&sh.hist[digit[j]], 1u);
    }
  }
  if (pass == 0 && saw_nonfinite) atomicOr(&F.flags[0], MST_FLAG_NONFINITE);
  __syncthreads();
  for (int b = threadIdx.x; b < BINS; b += FUSED_THREADS)
    if (sh.hist[b]) atomicAdd(&gh[b], sh.hist[b]);
}

// behind the barrier: every block picks the digit from the complete histogram (same arithmetic as the single-layer
// kernel) and advances the layer's selection state
template <int MODE>
__device__ void batch_hist_pick(const FusedParams& F, BatchLayerState& st, BatchShared& sh) {
  constexpr int KB = KeyBits<MODE>::value;
  const SelParams& P = F.sel;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int pass = st.pass;
  const int shift = pass_shift(KB, pass), width = pass_width(KB, pass);
  const unsigned long long prefix = st.prefix;
  const long long k = st.k;
  const int gpass = st.gpass;
  unsigned int* gh = F.hist + (gpass % 3) * BINS;
  unsigned int mine[FUSED_BPT];
  unsigned int tsum = 0;
#pragma unroll
  for (int j = 0; j < FUSED_BPT; ++j) {
    mine[j] = __ldcg(gh + threadIdx.x * FUSED_BPT + j);
    tsum += mine[j];
  }
  if (blockIdx.x == 0) {  // clear the buffer of pass gpass + 2 (last read before this barrier)
    unsigned int* gz = F.hist + ((gpass + 2) % 3) * BINS;
    for (int b = threadIdx.x; b < BINS; b += FUSED_THREADS) gz[b] = 0;
  }
  unsigned int incl = tsum;
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  __syncthreads();  // everyone has read the state; warp_tot is free
  if (threadIdx.x == 0) st.found = 0;
  if (lane == 31) sh.warp_tot[warp] = incl;
  __syncthreads();
  unsigned int before = incl - tsum;
  for (int wv = 0; wv < warp; ++wv) before += sh.warp_tot[wv];
  const bool owner = (long long)before < k && k <= (long long)before + (long long)tsum;
  if (owner) {
    long long cum = before;
    int bin = 0;
    unsigned int bcount = 0;
    for (int j = 0; j < FUSED_BPT; ++j) {
      if (cum + (long long)mine[j] >= k) { bin = j; bcount = mine[j]; break; }
      cum += mine[j];
    }
    const unsigned long long np = (prefix << width) | (unsigned long long)(threadIdx.x * FUSED_BPT + bin);
    st.prefix = np;
    st.k = k - cum;
    st.found = 1;
    if (shift == 0) {
      st.tau = np;
      st.rem = k - cum;
      st.need_rank = ((long long)bcount > k - cum) ? 1 : 0;
      st.done = 1;
    } else if ((long long)bcount == k - cum) {
      st.tau = (np << shift) | ((1ULL << shift) - 1ULL);
      st.rem = k - cum;
      st.need_rank = 0;
      st.done = 1;
    } else if (MODE == MODE_PRUNE && shift <= P.low_zero) {
      st.tau = np << shift;
      st.rem = k - cum;
      st.need_rank = 1;
      st.done = 1;
    }
  }
  __syncthreads();
  if (!st.found) {  // fewer candidates than requested (ruled out by the host counts): take everything
    __syncthreads();
    if (threadIdx.x == 0) {
      st.tau = ~0ULL;
      st.rem = 0x7FFFFFFFFFFFFFFFLL;
      st.need_rank = 0;
      st.done = 1;
      if (blockIdx.x == 0) atomicOr(&F.flags[0], MST_FLAG_CORRUPT);
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    st.gpass = gpass + 1;
    st.pass = pass + 1;
  }
  __syncthreads();
}

template <int MODE>
__device__ void batch_tie_count(const FusedParams& F, const BatchLayerState& st, const BatchSlice& sl, BatchShared& sh) {
  typedef typename KeyWord<MODE>::type K;
  const SelParams& P = F.sel;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const K tau = (K)st.tau;
  for (int64_t w = sl.lo + warp; w < sl.hi; w += FUSED_WARPS) {
    unsigned long long key64;
    bool nf;
    const bool c = cand_key_w<MODE>(P, w, lane, sl.s_old[w - sl.lo], sl.s_base[w - sl.lo], sl.s_grad[w - sl.lo], key64, nf);
    const unsigned eq = __ballot_sync(0xffffffffu, c && (K)key64 == tau);
    if (lane == 0) F.cnt[w] = __popc(eq);
  }
  __syncthreads();
  batch_scan_begin(F.cnt, sl.lo, sl.hi, F.bsums, st.gscan, sh.red);
}

template <int MODE>
__device__ void batch_mark(const FusedParams& F, const BatchLayerState& st, const BatchSlice& sl, uint32_t* out_bits) {
  typedef typename KeyWord<MODE>::type K;
  const SelParams& P = F.sel;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const K tau = (K)st.tau;
  const long long rem = st.rem;
  const bool need_rank = st.need_rank != 0;
  constexpr int MB = 4;
  for (int64_t w0 = sl.lo + warp; w0 < sl.hi; w0 += FUSED_WARPS * MB) {
    bool c[MB], iseq[MB];
    K key[MB];
#pragma unroll
    for (int j = 0; j < MB; ++j) {
      const int64_t w = w0 + (int64_t)j * FUSED_WARPS;
      bool nf = false;
      unsigned long long key64 = 0;
      const int64_t li = w < sl.hi ? w - sl.lo : 0;
      c[j] = w < sl.hi && cand_key_w<MODE>(P, w, lane, sl.s_old[li], sl.s_base[li], sl.s_grad[li], key64, nf);
      key[j] = (K)key64;
      iseq[j] = c[j] && key[j] == tau;
    }
#pragma unroll
    for (int j = 0; j < MB; ++j) {
      const int64_t w = w0 + (int64_t)j * FUSED_WARPS;
      if (w >= sl.hi) continue;  // uniform over the warp
      const unsigned eq = __ballot_sync(0xffffffffu, iseq[j]);
      const long long rank = need_rank ? (long long)F.scan[w] + __popc(eq & lanemask_lt()) : -1;
      const bool take = c[j] && (key[j] < tau || (iseq[j] && rank < rem));
      const unsigned bits = __ballot_sync(0xffffffffu, take);
      if (lane == 0) {
        out_bits[w] = bits;
        if (MODE == MODE_GRAD) sl.s_grad[w - sl.lo] = bits;  // the random selection of this block reads it from here
      }
    }
  }
  __syncthreads();
}

__device__ __forceinline__ long long batch_sel_count(const FusedParams& F, int sel) {
  return sel == 0 ? F.n_prune : (sel == 1 ? F.n_grad : F.n_rand);
}
__device__ __forceinline__ uint32_t* batch_sel_bits(const FusedParams& F, int sel) {
  return sel == 0 ? F.pruned_bits : (sel == 1 ? F.grad_bits : F.rand_bits);
}

// Non-barrier work until the layer reaches its next barrier phase: selections that take nothing write empty masks,
// the next selection with work gets its state, after the last one the mask rewrite is due.
__device__ void batch_advance(const FusedParams& F, BatchLayerState& st, const BatchSlice& sl) {
  __syncthreads();
  int sel = st.sel;
  while (sel <= 2 && batch_sel_count(F, sel) <= 0) {
    uint32_t* out = batch_sel_bits(F, sel);
    for (int64_t w = sl.lo + threadIdx.x; w < sl.hi; w += FUSED_THREADS) {
      out[w] = 0;
      if (sel == 1) sl.s_grad[w - sl.lo] = 0;
    }
    ++sel;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    st.sel = sel;
    if (sel <= 2) {
      st.prefix = 0;
      st.k = batch_sel_count(F, sel);
      st.tau = 0;
      st.rem = 0;
      st.need_rank = 0;
      st.done = 0;
      st.pass = 0;
      st.phase = PH_HIST;
    } else {
      st.phase = PH_REWRITE;
    }
  }
  __syncthreads();
}

__global__ void __launch_bounds__(FUSED_THREADS, 2) mg_update_batch_kernel(const BatchParams B) {
  cg::grid_group grid = cg::this_grid();
  __shared__ BatchShared sh;
  extern __shared__ uint32_t s_dyn[];
  mst_grid_launch_dependents();
  mst_grid_dependency_wait();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  BatchSlice sl[BATCH_MAX];
#pragma unroll
  for (int l = 0; l < BATCH_MAX; ++l) {
    if (l >= B.n) break;
    const SelParams& P = B.L[l].sel;
    const int64_t per = (P.nwords + gridDim.x - 1) / gridDim.x;
    sl[l].lo = per * blockIdx.x < P.nwords ? per * blockIdx.x : P.nwords;
    sl[l].hi = sl[l].lo + per < P.nwords ? sl[l].lo + per : P.nwords;
    sl[l].s_old = s_dyn + B.smem_off[l];
    sl[l].s_base = reinterpret_cast<int32_t*>(s_dyn + B.smem_off[l] + per);
    sl[l].s_grad = s_dyn + B.smem_off[l] + 2 * per;
    for (int64_t w = sl[l].lo + threadIdx.x; w < sl[l].hi; w += FUSED_THREADS) {
      sl[l].s_old[w - sl[l].lo] = P.old_bits[w];
      sl[l].s_base[w - sl[l].lo] = P.old_wscan[w];
      sl[l].s_grad[w - sl[l].lo] = 0;
    }
    if (threadIdx.x == 0) {
      sh.st[l].sel = 0;
      sh.st[l].phase = PH_NEW;
      sh.st[l].gpass = 0;
      sh.st[l].gscan = 0;
    }
  }
  __syncthreads();
  for (int l = 0; l < B.n; ++l) batch_advance(B.L[l], sh.st[l], sl[l]);

  for (;;) {
    // ---- work in front of the shared barrier
    bool pending = false;
    for (int l = 0; l < B.n; ++l) {
      const FusedParams& F = B.L[l];
      BatchLayerState& st = sh.st[l];
      const int phase = st.phase, sel = st.sel;   // uniform: written behind block barriers
      if (phase == PH_DONE) continue;
      pending = true;
      if (phase == PH_HIST) {
        if (sel == 0) batch_hist_sweep<MODE_PRUNE>(F, st, sl[l], sh);
        else if (sel == 1) batch_hist_sweep<MODE_GRAD>(F, st, sl[l], sh);
        else batch_hist_sweep<MODE_RAND>(F, st, sl[l], sh);
      } else if (phase == PH_TIE) {
        if (sel == 0) batch_tie_count<MODE_PRUNE>(F, st, sl[l], sh);
        else if (sel == 1) batch_tie_count<MODE_GRAD>(F, st, sl[l], sh);
        else batch_tie_count<MODE_RAND>(F, st, sl[l], sh);
      } else {  // PH_REWRITE: new = (old & ~pruned) | grad | rand, and its popcounts
        const SelParams& P = F.sel;
        for (int64_t w = sl[l].lo + threadIdx.x; w < sl[l].hi; w += FUSED_THREADS) {
          const uint32_t b = (P.old_bits[w] & ~F.pruned_bits[w]) | F.grad_bits[w] | F.rand_bits[w];
          F.new_bits[w] = b;
          F.cnt[w] = __popc(b);
        }
        __syncthreads();
        batch_scan_begin(F.cnt, sl[l].lo, sl[l].hi, F.bsums, st.gscan, sh.red);
      }
    }
    if (!pending) break;   // same decision in every block
    grid.sync();
    // ---- work behind it
    for (int l = 0; l < B.n; ++l) {
      const FusedParams& F = B.L[l];
      BatchLayerState& st = sh.st[l];
      const int phase = st.phase, sel = st.sel;
      if (phase == PH_DONE) continue;
      if (phase == PH_HIST) {
        constexpr int passes_mag = num_passes(32), passes_hash = num_passes(64);
        if (sel == 0) batch_hist_pick<MODE_PRUNE>(F, st, sh);
        else if (sel == 1) batch_hist_pick<MODE_GRAD>(F, st, sh);
        else batch_hist_pick<MODE_RAND>(F, st, sh);
        const bool finished = st.done || st.pass >= (sel == 2 ? passes_hash : passes_mag);
        if (!finished) continue;
        if (st.need_rank) {
          __syncthreads();
          if (threadIdx.x == 0) st.phase = PH_TIE;
          __syncthreads();
          continue;
        }
      } else if (phase == PH_TIE) {
        batch_scan_end(F.cnt, F.scan, F.sel.nwords, sl[l].lo, sl[l].hi, F.bsums, st.gscan, sh.red);
        __syncthreads();
        if (threadIdx.x == 0) st.gscan = st.gscan + 1;
        __syncthreads();
      } else {  // PH_REWRITE
        batch_scan_end(F.cnt, F.new_wscan, F.sel.nwords, sl[l].lo, sl[l].hi, F.bsums, st.gscan, sh.red);
        const SelParams& P = F.sel;
        for (int64_t w0 = sl[l].lo + warp; w0 < sl[l].hi; w0 += FUSED_WARPS * 4) {
          if (P.bf16)
            mst_fill_csr_words<uint16_t, 4>(w0, FUSED_WARPS, sl[l].hi, lane, F.new_bits, F.new_wscan, P.O, P.wpr, F.new_col,
                                            (uint16_t*)F.new_vals, F.new_row_ptr, P.old_bits, P.old_wscan,
                                            (const uint16_t*)P.vals, nullptr);
          else
            mst_fill_csr_words<float, 4>(w0, FUSED_WARPS, sl[l].hi, lane, F.new_bits, F.new_wscan, P.O, P.wpr, F.new_col,
                                         (float*)F.new_vals, F.new_row_ptr, P.old_bits, P.old_wscan, (const float*)P.vals,
                                         nullptr);
        }
        __syncthreads();
        if (threadIdx.x == 0) st.phase = PH_DONE;
        __syncthreads();
        continue;
      }
      // the selection is settled (threshold known, ties ranked if needed): mark it and move on
      if (sel == 0) batch_mark<MODE_PRUNE>(F, st, sl[l], F.pruned_bits);
      else if (sel == 1) batch_mark<MODE_GRAD>(F, st, sl[l], F.grad_bits);
      else batch_mark<MODE_RAND>(F, st, sl[l], F.rand_bits);
      __syncthreads();
      if (threadIdx.x == 0) {
        st.sel = sel + 1;
        st.phase = PH_NEW;
      }
      batch_advance(F, st, sl[l]);
    }
  }
}

inline unsigned long long host_mix(unsigned long long z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}

}  // namespace

extern "C" mst_status_t mst_update_counts(double prune_frac, int64_t nnz, int64_t target_nnz, int64_t numel,
                                          double random_ratio, int64_t counts[4]) {
  if (!counts) return MST_ERR_INVALID_ARG;
  if (!(prune_frac >= 0.0 && prune_frac <= 1.0) || !(random_ratio >= 0.0 && random_ratio <= 1.0))
    return MST_ERR_INVALID_ARG;
  if (nnz < 0 || nnz > numel) return MST_ERR_INVALID_ARG;
  if (target_nnz < 0) target_nnz = nnz;
  if (target_nnz > numel) return MST_ERR_INFEASIBLE;
  // floor(zeta * nnz) in double; then the smallest adjustment that lets the layer reach its target count
  int64_t n_prune = (int64_t)(prune_frac * (double)nnz);
  const int64_t lo = nnz - target_nnz > 0 ? nnz - target_nnz : 0;
  const int64_t hi = nnz < numel - target_nnz ? nnz : numel - target_nnz;
  if (n_prune < lo) n_prune = lo;
  if (n_prune > hi) n_prune = hi;
  const int64_t n_grow = n_prune + target_nnz - nnz;
  const int64_t n_rand = (int64_t)((double)n_grow * random_ratio);
  counts[0] = n_prune;
  counts[1] = n_grow;
  counts[2] = n_rand;
  counts[3] = n_grow - n_rand;
  return MST_OK;
}

extern "C" mst_status_t mst_rand_bracket(int64_t k, int64_t candidates, double sigmas, int64_t list_capacity, uint64_t* lo,
                                         uint64_t* hi, int32_t* planned) {
  if (!lo || !hi || !planned || list_capacity < 0) return MST_ERR_INVALID_ARG;
  *lo = *hi = 0;
  *planned = 0;
  if (k <= 0 || candidates <= 0 || k > candidates || !(sigmas > 0.0)) return MST_OK;   // nothing to bracket, or switched off
  const int64_t m = (int64_t)(sigmas * sqrt((double)k)) + 16;
  if (3 * m > list_capacity) return MST_OK;               // expected list length 2m: leave room for its own spread
  const int64_t lo_cnt = k - m > 0 ? k - m : 0, hi_cnt = k + m;
  const unsigned __int128 one = (unsigned __int128)1 << 64;
  const uint64_t l = (uint64_t)(one * (unsigned __int128)lo_cnt / (unsigned __int128)candidates);
  const uint64_t h = hi_cnt >= candidates ? ~(uint64_t)0 : (uint64_t)(one * (unsigned __int128)hi_cnt / (unsigned __int128)candidates);
  if (h <= l) return MST_OK;
  *lo = l;
  *hi = h;
  *planned = 1;
  return MST_OK;
}

namespace {

// One layer's update, planned on the host: counts, selection parameters, which buffer set is built.
struct UpdatePlan {
  mst_layer* L;
  int64_t n_prune, n_rand, n_grad, target;
  int c, n;  // live set, set being built
  SelParams P;
};

mst_status_t plan_update(mst_layer* L, double prune_frac, const mst_regrow_rule_t* rule, const float* G_dense, UpdatePlan* pl) {
  if (!L || !rule) return MST_ERR_INVALID_ARG;
  if (L->nnz < 0) return MST_ERR_NOT_PACKED;
  int64_t cnt[4];
  MST_TRY(mst_update_counts(prune_frac, L->nnz, rule->target_nnz, L->N, rule->random_ratio, cnt));
  pl->L = L;
  pl->n_prune = cnt[0];
  pl->n_rand = cnt[2];
  pl->n_grad = cnt[3];
  pl->target = rule->target_nnz < 0 ? L->nnz : rule->target_nnz;
  if (pl->target > L->cap) return MST_ERR_CAPACITY;
  if (!(rule->prune_grad_weight >= 0.f)) return MST_ERR_INVALID_ARG;
  if ((pl->n_grad > 0 || (rule->prune_grad_weight != 0.f && pl->n_prune > 0)) && !G_dense) return MST_ERR_INVALID_ARG;
  pl->c = L->cur;
  pl->n = L->cur ^ 1;
  SelParams& P = pl->P;
  P.old_bits = L->bits[pl->c];
  P.old_wscan = L->wscan[pl->c];
  P.vals = L->vals[pl->c];
  P.bf16 = L->dtype == MST_BF16;
  P.G = G_dense;
  P.pruned_bits = L->pruned_bits;
  P.grad_bits = L->grad_bits;
  P.O = L->O;
  P.I = L->I;
  P.wpr = L->wpr;
  P.allow = rule->allow_regrow_pruned ? 1 : 0;
  P.aligned = (L->I % 32 == 0) ? 1 : 0;
  P.lambda = rule->prune_grad_weight;
  P.low_zero = (L->dtype == MST_BF16 && P.lambda == 0.f) ? 16 : 0;
  P.nwords = L->nwords;
  {  // state of the random-growth generator for (seed, step, layer): three chained SplitMix64 first outputs
    const unsigned long long a = host_mix(rule->seed + SM64_GAMMA);
    const unsigned long long b = host_mix((a ^ rule->step) + SM64_GAMMA);
    P.stream = host_mix((b ^ (unsigned long long)(int64_t)L->layer_id) + SM64_GAMMA);
  }
  return MST_OK;
}

void fill_fused_params(const UpdatePlan& pl, FusedParams& F) {
  mst_layer* L = pl.L;
  const int n = pl.n;
  F.sel = pl.P;
  F.n_prune = pl.n_prune; F.n_grad = pl.n_grad; F.n_rand = pl.n_rand;
  F.pruned_bits = L->pruned_bits; F.grad_bits = L->grad_bits; F.rand_bits = L->rand_bits; F.new_bits = L->bits[n];
  F.cnt = L->word_cnt; F.scan = L->word_scan; F.bsums = L->block_sums;
  F.hist = L->hist; F.flags = L->flags;
  F.new_wscan = L->wscan[n]; F.new_row_ptr = L->row_ptr[n]; F.new_col = L->col_idx[n]; F.new_vals = L->vals[n];
  F.bitsT = L->bitsT; F.wscanT = L->wscanT; F.col_ptr = L->col_ptr; F.row_idx = L->row_idx; F.perm = L->perm;
  F.wpc = L->wpc; F.nwordsT = L->nwordsT;
  F.build_csc = mst_use_tensor_path(L) ? 0 : 1;
  F.smem_keys = 0;
  F.dual = 0;
  F.g_bulk = 0;
  F.rand_bracket = 0;
  F.rand_cap = L->rand_cap;
  F.rand_lo = F.rand_hi = 0;
  F.rand_list = L->rand_list;
  F.rand_ctr = L->rand_ctr;
}

// Bracket for the random growth: the n_rand-th smallest of C independent uniform 64-bit keys lies, with probability
// 1 - 1e-8 or better, between the quantiles (k - m) / C and (k + m) / C with m = sigmas * sqrt(k) + 16 (the count of
// keys below a quantile is binomial with a standard deviation below sqrt(k)).  The kernel checks the bracket against
// the exact counts and falls back to the general radix select when it missed, so the choice only affects speed.
void plan_rand_bracket(const UpdatePlan& pl, FusedParams& F) {
  const mst_layer* L = pl.L;
  double sigmas = 6.0;
  if (const char* e = getenv("MST_UPDATE_RAND_SIGMAS")) sigmas = atof(e);
  uint64_t lo = 0, hi = 0;
  int32_t planned = 0;
  // candidates: inactive entries the gradient growth left
  if (mst_rand_bracket(pl.n_rand, (L->N - L->nnz) - pl.n_grad, sigmas, L->rand_cap, &lo, &hi, &planned) != MST_OK || !planned) return;
  F.rand_lo = lo;
  F.rand_hi = hi;
  F.rand_bracket = 1;
}

// Host epilogue of an update whose kernels have been enqueued: statistics and error report when asked for, then the
// flip to the new buffer set.  `fused`: the structure was built by a fused kernel (single-layer or batched).
mst_status_t finish_update(const UpdatePlan& pl, bool fused, mst_update_stats_t* stats, cudaStream_t s) {
  mst_layer* L = pl.L;
  const int n = pl.n;
  const int64_t nnz_before = L->nnz;
  if (stats) {
    // the fused kernel records the longest row itself only when it also builds the CSC view
    if (!fused || !L->csc_valid) { max_row_nnz<<<(L->O + 255) / 256, 256, 0, s>>>(L->row_ptr[n], L->O, L->flags); MST_COUNT_LAUNCH(); }
    int32_t f[4] = {0, 0, 0, 0};
    int32_t total = 0;
    MST_CUDA_TRY(cudaMemcpyAsync(f, L->flags, sizeof(f), cudaMemcpyDeviceToHost, s));
    MST_CUDA_TRY(cudaMemcpyAsync(&total, L->wscan[n] + L->nwords, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    MST_CUDA_TRY(cudaStreamSynchronize(s));
    stats->nnz_before = nnz_before;
    stats->nnz_after = total;
    stats->n_prune = pl.n_prune;
    stats->n_grad = pl.n_grad;
    stats->n_rand = pl.n_rand;
    stats->max_row_nnz = f[1];
    const bool bad = (f[0] & (MST_FLAG_NONFINITE | MST_FLAG_CORRUPT)) || total != pl.target;
    if (bad) {
      // A rejected update is not applied: the structure built in the other buffer set is dropped and the layer keeps
      // its mask, values and nnz.  The CSC arrays may hold the rejected structure, so the view is rebuilt on next use.
      L->csc_valid = 0;
      MST_CUDA_TRY(cudaMemsetAsync(L->flags, 0, sizeof(int32_t), s));  // reported: cleared
      stats->nnz_after = nnz_before;
      return (f[0] & MST_FLAG_NONFINITE) ? MST_ERR_NONFINITE : MST_ERR_CORRUPT;
    }
  }
  L->cur = n;
  L->nnz = pl.target;
  ++L->version;
  if (!fused) MST_TRY(mst_build_csc(L, s));
  return MST_OK;
}

// grid of the fused kernels on the current device (0: cooperative launch unavailable)
int fused_grid_limit(const void* fn) {
  int dev = 0, coop = 0, sms = 0, occ = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, fn, FUSED_THREADS, 0) != cudaSuccess || !coop || occ < 1)
    return 0;
  if (occ > 2) occ = 2;
  return sms * occ;
}

mst_status_t launch_cooperative(const void* fn, void** args, int grid_blocks, size_t smem, cudaStream_t s) {
  // cooperative launch that may also start while its predecessor drains (the kernel waits before its first access)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid_blocks);
  cfg.blockDim = dim3(FUSED_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = mst_pdl_enabled() ? 2 : 1;
  if (getenv("MST_DEBUG")) fprintf(stderr, "libmst: cooperative launch grid %d block %d dynamic shared memory %zu\n", grid_blocks, FUSED_THREADS, smem);
  MST_CUDA_TRY(cudaLaunchKernelExC(&cfg, fn, args));
  MST_COUNT_LAUNCH();
  return MST_OK;
}

// kernels of one layer's update (everything except the host epilogue); *fused_out tells which form ran
mst_status_t launch_single_update(const UpdatePlan& pl, cudaStream_t s, bool* fused_out) {
  mst_layer* L = pl.L;
  const SelParams& P = pl.P;
  bool fused = true;
  if (const char* e = getenv("MST_UPDATE_FUSED")) fused = (e[0] != '0');
  int grid_blocks = 0;
  size_t fused_smem = 0;
  const void* fn = L->dtype == MST_F32 ? (const void*)mg_update_fused_kernel<float> : (const void*)mg_update_fused_kernel<uint16_t>;
  int smem_keys = 0;
  // Side-by-side selections: not with regrowth of just-pruned links (the gradient candidates then depend on the prune
  // result)
  bool want_dual = !P.allow;
  if (const char* e = getenv("MST_UPDATE_DUAL")) want_dual = want_dual && (e[0] != '0');
  if (fused) {
    grid_blocks = fused_grid_limit(fn);
    if (grid_blocks == 0) fused = false;
    else {
      const int64_t useful = (L->nwords + FUSED_WARPS - 1) / FUSED_WARPS;  // at least one word per warp
      if (grid_blocks > useful) grid_blocks = (int)(useful < 1 ? 1 : useful);
      int64_t per = (L->nwords + grid_blocks - 1) / grid_blocks;
      fused_smem = (size_t)per * 20;  // slice of mask, scan, grown, candidate and pruned words
      if ((per > (int64_t)FUSED_WARPS * KEYS_PER_LANE || want_dual) && !getenv("MST_UPDATE_NO_SMEM_KEYS")) {
        // keys in shared memory (128 bytes per mask word): always for the side-by-side form, otherwise when the
        // slice's keys do not fit the registers; if a block can have that much, with two blocks per SM or, for the
        // largest layers, one
        int dev = 0, sms = 0, optin = 0;
        if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) == cudaSuccess) {
          for (int occ_want = 2; occ_want >= 1 && !smem_keys; --occ_want) {
            int g = sms * occ_want;
            if (g > grid_blocks) g = grid_blocks;
            const int64_t per_k = (L->nwords + g - 1) / g;
            const size_t need = (size_t)per_k * (20 + 128);
            if (need + 10 * 1024 > (size_t)optin) continue;
            // never below the default limit: the attribute stays with the function, and a later launch that needs less
            // than 48 KiB does not set it again
            const size_t attr_bytes = need > 48 * 1024 ? need : 48 * 1024;
            if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attr_bytes) != cudaSuccess) continue;
            int occ = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, fn, FUSED_THREADS, need) != cudaSuccess || occ < 1) continue;
            if ((int64_t)occ * sms < g) continue;   // all blocks must be resident at once
            grid_blocks = g;
            per = per_k;
            fused_smem = need;
            smem_keys = 1;
          }
        }
      }
      // two alternating partial-sum areas of grid_blocks entries each (the buffer carries 1024 spare entries)
      if (2 * (int64_t)grid_blocks > mst_scan_block_sums_len(L->nwords > L->nwordsT ? L->nwords : L->nwordsT) + 1024) fused = false;
      if (!smem_keys && fused_smem > 36 * 1024) fused = false;  // very large layers: kernel-per-phase path
    }
  }
  if (fused) {
    // flags[0] (error bits) stays set until a reporting call has returned it; the kernel clears the per-update
    // statistics itself and leaves the histograms and the bracket counters zero for the next launch
    if (!L->scratch_clean) {
      MST_CUDA_TRY(cudaMemsetAsync(L->hist, 0, sizeof(unsigned int) * 3 * HSTRIDE, s));
      MST_CUDA_TRY(cudaMemsetAsync(L->rand_ctr, 0, 2 * sizeof(unsigned long long), s));
    }
    if (!mst_use_tensor_path(L)) MST_TRY(mst_alloc_csc(L));   // the kernel fills the view's arrays for such layers
    FusedParams F;
    fill_fused_params(pl, F);
    F.smem_keys = smem_keys;
    // the packed histogram of the side-by-side form needs fewer than 65536 entries per block
    const bool dual = want_dual && smem_keys && ((L->nwords + grid_blocks - 1) / grid_blocks) * 32 < 65536;
    F.dual = dual ? 1 : 0;
    F.g_bulk = (dual && P.aligned && P.G && ((uintptr_t)P.G % 16 == 0)) ? 1 : 0;
    if (dual) plan_rand_bracket(pl, F);
    L->csc_valid = F.build_csc;
    void* args[] = {&F};
    L->scratch_clean = 0;
    MST_TRY(launch_cooperative(fn, args, grid_blocks, fused_smem, s));
    L->scratch_clean = 1;
  } else {
    MST_CUDA_TRY(cudaMemsetAsync(L->flags + 1, 0, sizeof(int32_t) * 3, s));
    L->scratch_clean = 0;
    MST_TRY(run_select<MODE_PRUNE>(L, P, pl.n_prune, L->pruned_bits, s));
    MST_TRY(run_select<MODE_GRAD>(L, P, pl.n_grad, L->grad_bits, s));
    MST_TRY(run_select<MODE_RAND>(L, P, pl.n_rand, L->rand_bits, s));
    MST_TRY(mst_combine_update_bits(L, pl.n, s));
    MST_TRY(mst_rebuild_from_bits(L, pl.n, nullptr, 0, pl.c, s));
  }
  *fused_out = fused;
  return MST_OK;
}

}  // namespace

#ifdef MST_UPD_PROFILE
// (id, SM clock) pairs stamped by block 0 of the last fused update kernel; returns the number of pairs
extern "C" int mst_update_profile(long long* out, int max_pairs) {
  long long h[64];
  int n = 0;
  if (cudaDeviceSynchronize() != cudaSuccess || cudaMemcpyFromSymbol(h, g_upd_stamps, sizeof(h)) != cudaSuccess ||
      cudaMemcpyFromSymbol(&n, g_upd_nstamps, sizeof(int)) != cudaSuccess)
    return -1;
  if (n > max_pairs) n = max_pairs;
  for (int i = 0; i < 2 * n; ++i) out[i] = h[i];
  return n;
}
#endif

extern "C" mst_status_t mst_topology_update(mst_layer_t* L, double prune_frac, const mst_regrow_rule_t* rule,
                                            const float* G_dense, mst_update_stats_t* stats, mst_stream_t stream) {
  cudaStream_t s = (cudaStream_t)stream;
  UpdatePlan pl;
  MST_TRY(plan_update(L, prune_frac, rule, G_dense, &pl));
  bool fused = false;
  MST_TRY(launch_single_update(pl, s, &fused));
  return finish_update(pl, fused, stats, s);
}

extern "C" mst_status_t mst_topology_update_many(int32_t n_layers, mst_layer_t* const* layers, const double* prune_frac,
                                                 const mst_regrow_rule_t* rules, const float* const* G_dense,
                                                 mst_update_stats_t* stats, mst_stream_t stream) {
  if (n_layers < 0 || (n_layers > 0 && (!layers || !prune_frac || !rules || !G_dense))) return MST_ERR_INVALID_ARG;
  if (n_layers == 0) return MST_OK;
  cudaStream_t s = (cudaStream_t)stream;
  // every layer is validated before anything is launched: an argument error leaves all layers untouched
  UpdatePlan* plans = new (std::nothrow) UpdatePlan[n_layers];
  char* mode = new (std::nothrow) char[n_layers];   // 0: not launched yet, 1: batched, 2: single fused, 3: kernel per phase
  if (!plans || !mode) { delete[] plans; delete[] mode; return MST_ERR_INVALID_ARG; }
  mst_status_t st = MST_OK;
  for (int i = 0; i < n_layers && st == MST_OK; ++i) {
    st = plan_update(layers[i], prune_frac[i], &rules[i], G_dense[i], &plans[i]);
    mode[i] = 0;
    for (int j = 0; j < i && st == MST_OK; ++j)
      if (layers[j] == layers[i]) st = MST_ERR_INVALID_ARG;   // a layer may appear once
  }
  const int grid_limit = st == MST_OK ? fused_grid_limit((const void*)mg_update_batch_kernel) : 0;
  // Measured on GPT-2 shapes: a layer whose keys fit the single-layer kernel's register or shared-memory cache
  // (every layer up to GPT-2 large) is updated faster on its own (0.42 ms for the four layers of a GPT-2-medium block)
  // than in a shared launch, which has to recompute its keys in every pass (0.56 ms).  The shared launch is therefore
  // off unless MST_UPDATE_BATCH=1 asks for it.
  bool batching = false;
  if (const char* e = getenv("MST_UPDATE_BATCH")) batching = grid_limit > 0 && (e[0] == '1');
  int i = 0;
  while (st == MST_OK && i < n_layers) {
    // collect the next run of layers that can share a launch: tensor-path layers (no CSC view to build) whose slices
    // fit shared memory together and whose scan scratch holds two partial-sum areas of the grid
    BatchParams B;
    B.n = 0;
    size_t words = 0;
    int first = i;
    while (batching && i < n_layers && B.n < BATCH_MAX) {
      mst_layer* L = plans[i].L;
      const size_t per = (size_t)((L->nwords + grid_limit - 1) / grid_limit);
      const bool ok = mst_use_tensor_path(L) && 2 * (int64_t)grid_limit <= mst_scan_block_sums_len(L->nwords) + 1024 &&
                      (words + 3 * per) * 4 <= 40 * 1024;
      if (!ok) break;
      B.smem_off[B.n] = (int)words;
      words += 3 * per;
      fill_fused_params(plans[i], B.L[B.n]);
      B.L[B.n].build_csc = 0;
      ++B.n;
      ++i;
    }
    if (B.n >= 2) {
      for (int j = first; j < i && st == MST_OK; ++j) {
        mst_layer* L = plans[j].L;
        if (cudaMemsetAsync(L->flags + 1, 0, sizeof(int32_t) * 3, s) != cudaSuccess ||
            cudaMemsetAsync(L->hist, 0, sizeof(unsigned int) * 3 * BINS, s) != cudaSuccess)
          st = MST_ERR_CUDA;
        L->csc_valid = 0;
        L->scratch_clean = 0;
        mode[j] = 1;
      }
      if (st == MST_OK) {
        void* args[] = {&B};
        st = launch_cooperative((const void*)mg_update_batch_kernel, args, grid_limit, words * 4, s);
      }
    } else {
      // a run of one (or a layer that cannot be batched): the single-layer path
      i = first;
      bool fused = false;
      st = launch_single_update(plans[i], s, &fused);
      mode[i] = fused ? 2 : 3;
      ++i;
    }
  }
  // host epilogues in order; the first failure is reported, later layers are still finished so that no layer is left
  // with kernels enqueued but its buffer sets not flipped
  for (int j = 0; j < n_layers; ++j) {
    if (mode[j] == 0) continue;
    const mst_status_t fj = finish_update(plans[j], mode[j] != 3, stats ? &stats[j] : nullptr, s);
    if (st == MST_OK) st = fj;
  }
  delete[] plans;
  delete[] mode;
  return st;
}
