/*
 * libmst: the unstructured-sparse fully-connected layer of Mixed Sparsity Training
 * (arXiv 2408.11746) for NVIDIA B200 (sm_100a).
 *
 * One handle = one layer theta_l [O x I] (out_features x in_features, row-major, PyTorch layout)
 * under a binary mask M (Sec. 3.2).  The layer is stored as canonical CSR (columns ascending in
 * each row) plus a CSC view; the flat index of entry (o, i) is o*I + i.
 *
 * Conventions for every call
 *   - returns mst_status_t; nothing throws, aborts, traps or spins without bound.
 *   - every pointer named "device" is a CUDA device pointer owned by the caller; the handle owns
 *     its sparse arrays and its scratch, sized once for nnz_capacity (never reallocated).
 *   - leading dimensions (ld*) are in elements; activations are row-major [tokens x features].
 *   - element type of X, Y, dY, dX, W and the stored values is the layer's dtype
 *     (MST_F32: float; MST_BF16: 16-bit bfloat16 patterns); accumulation is always fp32.
 *   - work is enqueued on the caller's stream and is stream-ordered; calls that return data to
 *     host memory (stats, nnz) synchronise that stream.
 *   - argument, shape, dtype, capacity and count errors are detected on the host before any
 *     launch.  Problems only the device can see (a non-finite selection key, a corrupt structure)
 *     set a flag in handle-owned memory that stays set until mst_validate or
 *     mst_topology_update(stats != NULL) has returned it once; an update with stats == NULL
 *     never clears it.
 *   - calls that split their contraction range (mst_dense_grad, mst_dense_grad_dw, mst_sddmm_dw,
 *     mst_layer_step_host[_async] on bf16 layers) keep partial sums in one scratch buffer per
 *     device, allocated on first use and grown on demand: two such calls must not overlap on the
 *     GPU (one stream, or ordered by events).
 */
#ifndef MST_H_
#define MST_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mst_layer mst_layer_t;
typedef void* mst_stream_t; /* a cudaStream_t; NULL = the default stream */

typedef enum { MST_F32 = 0, MST_BF16 = 1 } mst_dtype_t;

typedef enum {
  MST_OK = 0,
  MST_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, value outside its range          */
  MST_ERR_SHAPE = 2,       /* leading dimension smaller than the row, feature count > 65535   */
  MST_ERR_DTYPE = 3,       /* unknown dtype                                                   */
  MST_ERR_CAPACITY = 4,    /* nnz (or target nnz) exceeds the capacity given at creation      */
  MST_ERR_INFEASIBLE = 5,  /* no prune/grow counts satisfy the request                        */
  MST_ERR_NONFINITE = 6,   /* Inf/NaN met in |w| or |g| while selecting                       */
  MST_ERR_CORRUPT = 7,     /* sparse structure fails validation                               */
  MST_ERR_CUDA = 8,        /* a CUDA runtime call failed                                      */
  MST_ERR_NOT_PACKED = 9   /* the layer has no structure yet (call mst_pack first)            */
} mst_status_t;

/* Growth rule of one topology update (Algorithm 1; Table "Comparison of different topology evolution schemes").
 *   target_nnz          active entries after the update, (1 - s_l') N_l; < 0 keeps the current count
 *   random_ratio        R in [0,1], share of grown links drawn at random (0 = RigL rule, 1 = SET rule)
 *   seed, step          the random-growth ranking is a pure function of (seed, step, layer_id, flat index):
 *                       candidates are ranked by SplitMix64 outputs (smaller first, ties by flat index)
 *   allow_regrow_pruned 0: links pruned in this update are not candidates for growth (default reading);
 *                       1: gradient growth may also pick just-pruned links (such a link keeps its value)
 *   prune_grad_weight   lambda >= 0 of the MEST pruning criterion |theta| + lambda |grad| (scheme table); 0 = prune by
 *                       |theta| alone (Mixed-Growing, SET, RigL).  With lambda != 0 the key is formed in fp32, one
 *                       rounding per operation, and G_dense is needed even when nothing grows by gradient */
typedef struct {
  int64_t target_nnz;
  double random_ratio;
  uint64_t seed;
  uint64_t step;
  int32_t allow_regrow_pruned;
  float prune_grad_weight;
} mst_regrow_rule_t;

typedef struct {
  int64_t nnz_before, nnz_after, n_prune, n_grad, n_rand, max_row_nnz;
} mst_update_stats_t;

/* Create an empty layer.  out_features, in_features in [1, 65535]; nnz_capacity in [1, O*I].
 * Allocates all device memory the layer will ever use on the current device. */
mst_status_t mst_layer_create(mst_layer_t** layer, int32_t layer_id, int32_t out_features, int32_t in_features,
                              mst_dtype_t dtype, int64_t nnz_capacity);
mst_status_t mst_layer_destroy(mst_layer_t* layer);

/* Which kernels serve forward, input gradient and weight gradient of a bf16 layer:
 *   MST_PATH_CUDA_CORE    the sparse kernels (work proportional to nnz, fp32 FMA pipe)
 *   MST_PATH_TENSOR_CORE  dense-tile kernels: W.M is expanded on the fly to a dense bf16 image and contracted on the
 *                         tensor cores (work proportional to O*I, about 18x the FMA pipe's rate); the weight gradient
 *                         is the dense contraction sampled on the mask in its epilogue.  Needs 16-byte-aligned rows
 *                         (leading dimensions multiple of 8), otherwise the CUDA-core kernels are used.
 *   MST_PATH_SPARSE_TC    forward and input gradient on the 2:4 structured-sparse tensor-core instruction: W.M is
 *                         split into the first two entries of every group of four consecutive contraction indices
 *                         (run at twice the dense tensor rate) and the few third and fourth entries, which the
 *                         kernel's epilogue adds from a feature-major copy of the activation columns they multiply.
 *                         Exact for any mask; pays off while few groups hold more than two entries (density up to
 *                         about 0.25).  Needs nnz <= O*I/4 and aligned operands, otherwise the dense tiles are used.
 *                         The weight gradient stays the dense contraction sampled on the mask.
 *   MST_PATH_AUTO         (default) bf16 layers with aligned operands: the structured-sparse instruction at densities
 *                         where it was measured faster than dense tiles, dense tiles above; CUDA cores otherwise.
 * fp32 layers always use the CUDA-core kernels.  Results of the paths agree within the stated tolerance, not
 * bit for bit (different summation order). */
typedef enum { MST_PATH_AUTO = 0, MST_PATH_CUDA_CORE = 1, MST_PATH_TENSOR_CORE = 2, MST_PATH_SPARSE_TC = 3 } mst_compute_path_t;
mst_status_t mst_set_compute_path(mst_layer_t* layer, mst_compute_path_t path);

/* The kernels forward and input gradient of this layer run on for aligned operands, with MST_PATH_AUTO resolved
 * (unaligned operands always fall back to the CUDA-core kernels). */
mst_status_t mst_layer_path_in_use(const mst_layer_t* layer, mst_compute_path_t* path);

/* Kernels the library has enqueued in this process so far (all layers, all streams): for launch accounting. */
mst_status_t mst_launch_count(int64_t* count);

/* Number of active entries (host value; known after mst_pack / mst_topology_update without a sync). */
mst_status_t mst_layer_nnz(const mst_layer_t* layer, int64_t* nnz);

/* Dense mask -> sparse structure (Sec. 3.2: the binary mask M_theta; Algorithm 1: theta <- theta . M).
 *   W_dense  device, [O x ldw] in the layer's dtype; only entries under the mask are read
 *   mask     device, uint8 [O x I] contiguous, non-zero = active
 * Builds CSR, the CSC view and the bit mask.  Synchronises the stream (returns nnz to the host);
 * MST_ERR_CAPACITY if the mask holds more than nnz_capacity entries (layer left unpacked). */
mst_status_t mst_pack(mst_layer_t* layer, const void* W_dense, int64_t ldw, const uint8_t* mask, mst_stream_t stream);

/* Canonical CSR out: row_ptr int32 [O+1], col_idx int32 [nnz], vals [nnz] in the layer's dtype; all device,
 * any of the three may be NULL to skip it. */
mst_status_t mst_export_csr(const mst_layer_t* layer, int32_t* row_ptr, int32_t* col_idx, void* vals,
                            mst_stream_t stream);
/* CSC view out: col_ptr int32 [I+1], row_idx int32 [nnz] (rows ascending in each column),
 * perm int32 [nnz] = CSR position of each CSC entry; device; any may be NULL. */
mst_status_t mst_export_csc(const mst_layer_t* layer, int32_t* col_ptr, int32_t* row_idx, int32_t* perm,
                            mst_stream_t stream);

/* Device pointer to the stored values (CSR order, layer dtype) so an optimizer can update them in place.
 * The pointer changes at every mst_pack / mst_topology_update. */
mst_status_t mst_values(mst_layer_t* layer, void** vals, int64_t* nnz);

/* Value tracking.  By default the library assumes that the stored values may have been modified in place before any
 * call, and rebuilds what it derives from them (the dense image of W.M for the tensor-core kernels, the compressed
 * operand of the structured-sparse path) at every forward and input-gradient call.  mst_track_values(layer, 1) is the
 * caller's promise to call mst_values_changed(layer) after every in-place modification (an optimizer step); the
 * derived operands are then rebuilt only when the mask or the values have changed since they were built, e.g. once
 * per training step instead of once per product.  mst_pack and mst_topology_update announce their own changes. */
mst_status_t mst_track_values(mst_layer_t* layer, int32_t enable);
mst_status_t mst_values_changed(mst_layer_t* layer);

/* Structure check on the device: row pointers monotone and ending at nnz, columns in range and strictly
 * ascending, CSC consistent with CSR, bit mask consistent.  Synchronises.  MST_ERR_CORRUPT / MST_ERR_NONFINITE
 * (sticky flag from an earlier update) or MST_OK. */
mst_status_t mst_validate(const mst_layer_t* layer, mst_stream_t stream);

/* Forward, Y[t,o] = sum_{i:(o,i) in M} W[o,i] X[t,i]   (Algorithm 1: the layer computes with theta . M; no bias;
 * cost (1-S)(2I-1)O per token, Eq. (3)).  X device [T x ldx], Y device [T x ldy]. */
mst_status_t mst_spmm_fwd(const mst_layer_t* layer, const void* X, int64_t ldx, int64_t T, void* Y, int64_t ldy,
                          mst_stream_t stream);

/* Input gradient, dX[t,i] = sum_{o:(o,i) in M} dY[t,o] W[o,i]   (App. "FLOP Calculation": backward = 2 x forward).
 * dY device [T x lddy], dX device [T x lddx].  Uses the CSC view: a gather, no floating-point atomics. */
mst_status_t mst_spmm_bwd_x(const mst_layer_t* layer, const void* dY, int64_t lddy, int64_t T, void* dX, int64_t lddx,
                            mst_stream_t stream);

/* First layer of the MLP with its activation fused behind the product: H = GELU(X (W.M)^T), GELU(y) = y Phi(y)
 * with Phi the standard normal distribution function (App. "Hyperparameters": activation GELU, no bias; the MLP
 * term FLOPs_MLP of the FLOP model is fc1 -> GELU -> fc2).  X device [T x ldx]; H device [T x ldh], layer dtype.
 * Y_pre (device [T x ldpre], layer dtype) receives the pre-activation X (W.M)^T for the backward pass; NULL to
 * skip it.  On the tensor path GELU is taken on the fp32 accumulator, before the rounding to bf16. */
mst_status_t mst_spmm_fwd_gelu(const mst_layer_t* layer, const void* X, int64_t ldx, int64_t T, void* Y_pre,
                               int64_t ldpre, void* H, int64_t ldh, mst_stream_t stream);

/* Input gradient of the second MLP layer carried through the activation in one pass:
 * dPre[t,i] = (sum_{o:(o,i) in M} dY[t,o] W[o,i]) * GELU'(Y_pre[t,i]),  GELU'(y) = Phi(y) + y phi(y)
 * (same passages; chain rule through H = GELU(Y_pre)).  `layer` is the layer that consumed H (fc2), so Y_pre and
 * dPre have in_features columns: Y_pre device [T x ldpre] (read only), dPre device [T x lddpre], layer dtype. */
mst_status_t mst_spmm_bwd_x_gelu(const mst_layer_t* layer, const void* dY, int64_t lddy, int64_t T, const void* Y_pre,
                                 int64_t ldpre, void* dPre, int64_t lddpre, mst_stream_t stream);

/* Unfactorized strided sparse self-attention, forward (Sec. 3.3):
 *   Out[i] = sum_{j in S_i} softmax_j(q_i . k_j / sqrt(d)) v_j,   S_i = { j <= i : i - j < l  or  (i - j) mod l == 0 },
 * the same S_i in every head (the set formula is printed with an intersection; text, figure and the FLOP ratios of
 * the appendix table fix the union).  Q, K, V: device bf16, token-major, `ld` elements between consecutive tokens,
 * head h in columns h*head_dim .. (so the three column slices of a fused qkv activation can be passed as they are);
 * token b*seq_len + i is position i of sequence b.  Out: device bf16 [batch*seq_len x ldo], same column layout.
 * lse (device float [batch, heads, seq_len], may be NULL) receives log sum_j exp(q_i . k_j / sqrt(d)) for a backward
 * pass.  Supported: head_dim = 64, seq_len a multiple of 128, stride l a positive multiple of 64, ld and ldo
 * multiples of 8, 16-byte aligned pointers; anything else MST_ERR_SHAPE.  Scores and sums are fp32, the softmax
 * weights are rounded to bf16 before they multiply the values.  Two kernels serve the call (a tcgen05 one for
 * l = 256 with seq_len <= 8 l, a warp-level one for everything else); which one runs does not change the contract. */
mst_status_t mst_strided_attention_fwd(const void* Q, const void* K, const void* V, int64_t ld, int32_t batch,
                                       int32_t seq_len, int32_t heads, int32_t head_dim, int32_t stride, void* Out,
                                       int64_t ldo, float* lse, mst_stream_t stream);

/* Backward of mst_strided_attention_fwd (same passage; the derivative of the definition above):
 *   delta_i = dOut_i . Out_i,  P_ij = exp(q_i . k_j / sqrt(d) - lse_i),  dS_ij = P_ij (dOut_i . v_j - delta_i),
 *   dV_j = sum_i P_ij dOut_i,  dK_j = sum_i dS_ij q_i / sqrt(d),  dQ_i = sum_j dS_ij k_j / sqrt(d)   (sums over the pairs
 *   with j in S_i).
 * Q, K, V, ld as in the forward call; Out [batch*seq_len x ldo] the forward output, dOut [batch*seq_len x lddo] the
 * upstream gradient, lse [batch, heads, seq_len] the forward's log-sum-exp (all device, bf16 except lse).
 * dQ, dK, dV: device bf16, ldg elements between tokens, head h in columns h*head_dim .. (three column slices of one
 * fused gradient buffer may be passed).  Supported: head_dim = 64, seq_len and stride multiples of 64, leading
 * dimensions multiples of 8, 16-byte aligned pointers; anything else MST_ERR_SHAPE.  Deterministic (no atomics).
 * Keeps one float per (token, head) in a per-device scratch buffer: calls must not overlap on the GPU. */
mst_status_t mst_strided_attention_bwd(const void* Q, const void* K, const void* V, int64_t ld, const void* Out,
                                       int64_t ldo, const void* dOut, int64_t lddo, const float* lse, int32_t batch,
                                       int32_t seq_len, int32_t heads, int32_t head_dim, int32_t stride, void* dQ,
                                       void* dK, void* dV, int64_t ldg, mst_stream_t stream);

/* Weight gradient on the mask only, dW[k] = sum_t dY[t,o_k] X[t,i_k] for the k-th active entry in CSR order
 * (same passage).  dW_vals device float [nnz].  May use the per-device split scratch (see the conventions above). */
mst_status_t mst_sddmm_dw(const mst_layer_t* layer, const void* dY, int64_t lddy, const void* X, int64_t ldx, int64_t T,
                          float* dW_vals, mst_stream_t stream);

/* Dense gradient for growth, G = dY^T X, float [O x I] contiguous (Algorithm 1, gradient-growth line: |grad L| on
 * empty slots; Sec. 2.1 "infrequent full gradient calculation").  No layer handle: a plain contraction.
 * bf16 inputs with 16-byte-aligned rows run on the tensor cores and may use a process-wide scratch buffer for
 * split partial sums (allocated on first use, grown on demand): such calls must not overlap on the GPU. */
mst_status_t mst_dense_grad(const void* dY, int64_t lddy, const void* X, int64_t ldx, int64_t T, int32_t out_features,
                            int32_t in_features, mst_dtype_t dtype, float* G, mst_stream_t stream);

/* Weight gradient on the mask read out of a dense gradient: dW[k] = G[o_k, i_k] (CSR order).  On steps that compute
 * the dense gradient anyway (every topology-update step: Algorithm 1 needs |grad L| on the empty slots and the
 * optimizer needs it on the active ones) the separate SDDMM contraction is redundant.
 * mst_dense_grad_dw = mst_dense_grad followed by this sampling: both G [O x I] and dW_vals [nnz] are written. */
mst_status_t mst_sddmm_from_dense(const mst_layer_t* layer, const float* G_dense, float* dW_vals, mst_stream_t stream);
mst_status_t mst_dense_grad_dw(const mst_layer_t* layer, const void* dY, int64_t lddy, const void* X, int64_t ldx,
                               int64_t T, float* G_dense, float* dW_vals, mst_stream_t stream);

/* Counts of one update (Algorithm 1, count lines), as the library computes them on the host:
 *   n_prune = clamp(floor(prune_frac * nnz), max(0, nnz - target), min(nnz, N - target)),
 *   n_grow = n_prune + target - nnz, n_rand = floor(n_grow * R), n_grad = n_grow - n_rand.
 * counts = {n_prune, n_grow, n_rand, n_grad}. */
mst_status_t mst_update_counts(double prune_frac, int64_t nnz, int64_t target_nnz, int64_t numel, double random_ratio,
                               int64_t counts[4]);

/* Planning helper of the random growth (host only, no device work).  The hash keys of the `candidates` entries that may
 * be grown at random are independent and uniform over 64 bits, so the k-th smallest of them lies, with probability
 * 1 - 1e-8 or better at sigmas = 6, in [lo, hi) = [(k - m) / candidates, (k + m) / candidates) * 2^64 with
 * m = sigmas * sqrt(k) + 16 (the count of keys below a quantile is binomial with a standard deviation below sqrt(k)).
 * The update kernel lists the about 2m candidates inside the bracket and finds the threshold among them; it checks the
 * bracket against the exact counts and falls back to a general selection when it missed, so the bracket affects
 * speed only.  *planned = 0 (and lo = hi = 0) when there is nothing to bracket (k <= 0, k > candidates), sigmas <= 0,
 * or 3m exceeds list_capacity, the number of candidates the layer's list can hold. */
mst_status_t mst_rand_bracket(int64_t k, int64_t candidates, double sigmas, int64_t list_capacity, uint64_t* lo,
                              uint64_t* hi, int32_t* planned);

/* One Mixed-Growing topology update (Algorithm 1): prune the n_prune active entries of smallest |w|, grow the n_grad
 * empty slots of largest |g| and n_rand more at random, rewrite the mask, drop pruned values, start grown values at
 * +0.0, rebuild CSR/CSC in place.  Ties are broken by the smaller flat index.  Selection is bit-exact and
 * deterministic.
 *   prune_frac  zeta in [0,1]
 *   G_dense     device float [O x I] contiguous; may be NULL iff n_grad == 0
 *   stats       host, may be NULL; when given the call synchronises and reports device-side errors.  An update that
 *               is reported as failed (MST_ERR_NONFINITE, MST_ERR_CORRUPT) is NOT applied: mask, values and nnz stay
 *               as they were.  With stats == NULL nothing is checked on the host: a non-finite key then leaves an
 *               applied, undefined selection behind and the error flag set for the next reporting call. */
mst_status_t mst_topology_update(mst_layer_t* layer, double prune_frac, const mst_regrow_rule_t* regrow_rule,
                                 const float* G_dense, mst_update_stats_t* stats, mst_stream_t stream);

/* The same update for several layers in one call (in training all layers are updated on the same step): identical
 * results, bit for bit, to calling mst_topology_update on each layer in turn.  prune_frac[i], rules[i], G_dense[i]
 * belong to layers[i]; stats is NULL or an array of n_layers entries (same meaning as above, the call then
 * synchronises once per layer).  A layer may appear once.  All arguments are validated before anything is launched.
 * With MST_UPDATE_BATCH=1 in the environment up to 8 tensor-path layers share one cooperative launch and its grid-wide
 * barriers; measured slower than one launch per layer on GPT-2 shapes (the shared launch cannot keep the layers'
 * keys on chip between passes), so it is off by default.
 * Returns the first error met; layers before and after it are still completed. */
mst_status_t mst_topology_update_many(int32_t n_layers, mst_layer_t* const* layers, const double* prune_frac,
                                      const mst_regrow_rule_t* rules, const float* const* G_dense,
                                      mst_update_stats_t* stats, mst_stream_t stream);

/* One training step of the layer from HOST buffers (pinned memory recommended): copies X [T x I] and dY [T x O]
 * (contiguous, layer dtype) to the device, runs forward, input gradient and weight gradient, and copies
 * Y [T x O], dX [T x I] (layer dtype) and dW_vals float [nnz] back.  Any output may be NULL to skip its copy.
 * Staging buffers live in the handle and grow on demand.  Synchronises the stream. */
mst_status_t mst_layer_step_host(mst_layer_t* layer, const void* X_host, const void* dY_host, int64_t T, void* Y_host,
                                 void* dX_host, float* dW_vals_host, mst_stream_t stream);

/* Dense mask -> canonical CSR with no handle and NO allocation (the paper has no counterpart: this entry point
 * exists for callers that must not allocate device memory).
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a host framework that has handed the whole GPU to its
 * own memory pool and forbids plugins to allocate, a real-time or serving loop that must not take the allocator's
 * implicit device synchronisation, or a thread working while another thread of the process is capturing a stream
 * (allocation calls are illegal during a global-mode capture).  Those callers cannot create an mst_layer_t (creation
 * allocates), yet still want the compressed structure of a mask.
 *
 * Same result as mst_pack followed by mst_export_csr, written into the caller's buffers:
 *   W_dense  device, [O x ldw] layer dtype;  mask device uint8 [O x I]
 *   row_ptr  device int32 [O+1]; row_ptr[O] receives the true number of active entries
 *   col_idx  device int32 [nnz_capacity];  vals device [nnz_capacity] in `dtype`
 * Entries at CSR positions >= nnz_capacity are not written (compare row_ptr[O] with the capacity afterwards).
 * Work space is a fixed array inside the library (about 3 MB of device memory on every GPU that loads the library,
 * held until the process ends), which limits the layer to O*I <= 4 194 304 entries and O*ceil(I/32) <= 262 144 mask
 * words; larger layers return MST_ERR_CAPACITY.  The call itself allocates nothing and frees nothing.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress); make that first call
 * outside any stream capture.  All calls share the one array: calls whose GPU work may overlap (different streams,
 * different threads) race on it - keep them on one stream or order them with events.  Nothing in the array has to
 * be cleared between calls; every call overwrites the part it reads.  Asynchronous on `stream`. */
mst_status_t mst_mask_to_csr_noalloc(int32_t out_features, int32_t in_features, mst_dtype_t dtype, const void* W_dense,
                                     int64_t ldw, const uint8_t* mask, int64_t nnz_capacity, int32_t* row_ptr,
                                     int32_t* col_idx, void* vals, mst_stream_t stream);

/* ---- Sparsity-Variation driver (host scalars; Sec. 3.1 equations for S_t, Sec. 3.2 for zeta_t and the Erdos-Renyi
 * split; Table "Private hyperparameters of MST": S_M = 0.96, N = 5, Delta_W = Delta_R = 2000, T_U = 100000,
 * zeta_1 = 0.3).  The printed equations are garbled; the reading is the cited cubic schedule, stepwise per stage:
 *   warm-up      t in [0, N*delta_w):           S_t = S_M * (1 - (1 - k/N)^3),  k = floor(t / delta_w)
 *   ultra-sparse t in [T_W, T_W + t_ultra):     S_t = S_M
 *   restoration  t' = t - T_W - T_U in [0, N*delta_r):  S_t = S_M * (1 - k/N)^3,  k = floor(t' / delta_r); then 0.
 * zeta_t = zeta_i / 2 * (1 + cos(pi (t - T_{i-1}) / (T_i - T_{i-1}))) on [T_{i-1}, T_i), T_0 = 0, T_1 = T_W + T_U,
 * T_{i+1} = T_i + delta_r; zeta_i = zeta_1 * decay^(i-1) (the paper gives only zeta_1; decay = 1: no decay).
 * mst_er_densities: d_l = eps (I_l + O_l) / (I_l O_l), eps such that sum d_l O_l I_l = global_density * sum O_l I_l;
 * layers that would exceed 1 become dense and eps is re-solved. */
typedef struct {
  double max_sparsity; /* S_M */
  int32_t n_stages;    /* N */
  int64_t delta_w;     /* pruning frequency, steps per warm-up stage */
  int64_t t_ultra;     /* T_U */
  int64_t delta_r;     /* growing frequency, steps per restoration stage */
} mst_sv_schedule_t;
mst_status_t mst_sv_sparsity(const mst_sv_schedule_t* schedule, int64_t step, double* sparsity);
mst_status_t mst_sv_update_fraction(const mst_sv_schedule_t* schedule, int64_t step, double zeta1, double decay,
                                    double* zeta);
mst_status_t mst_er_densities(int32_t n_layers, const int32_t* out_features, const int32_t* in_features,
                              double global_density, double* densities);

/* Sticky error bits of kernels that run without a layer handle (bit 0: a bounded wait inside the tensor-core
 * contraction expired and the block gave up; its output is then undefined; bit 1: the same in the attention
 * kernel; bit 2: the same in the structured-sparse contraction;
 * bit 3: the same in the CUDA-core SpMM / SDDMM).  Synchronises the device. */
mst_status_t mst_device_error_flags(int32_t* flags);

/* The same step without the final wait: inputs are copied on a copy-in stream owned by the layer, the three products
 * run on `stream`, results are copied back on a copy-out stream owned by the layer.  Calls for several layers issued
 * one after the other overlap one layer's copies with another layer's kernels (host buffers must be pinned for that).
 * mst_layer_step_host_wait blocks until the results of the layer's latest async step (and of every earlier one) are
 * in host memory.  Steps of one layer may be issued back to back without a wait: the next step's inputs are copied in
 * once the previous step's kernels have read them, its kernels start once the previous results have left the device
 * buffers; the host buffers of a step must stay untouched until a wait that covers it has returned. */
mst_status_t mst_layer_step_host_async(mst_layer_t* layer, const void* X_host, const void* dY_host, int64_t T,
                                       void* Y_host, void* dX_host, float* dW_vals_host, mst_stream_t stream);
mst_status_t mst_layer_step_host_wait(mst_layer_t* layer);

const char* mst_status_string(mst_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* MST_H_ */
