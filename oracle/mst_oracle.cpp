// CPU checker for the masked fully-connected layer of Mixed Sparsity Training.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference the CUDA
// library is compared against.  It shares no code with the CUDA path and the
// product never calls it.
//
// Everything is written on the paper's own data structure: a dense weight
// array theta [O x I] and a dense binary mask M [O x I] (Sec. 3.2: the binary
// mask that outlines the sparse topology).  Floating point is fp64.
//
//   forward          Y  = X (theta . M)^T          Algorithm 1 (theta <- theta . M), Eq. (3) cost model
//   input gradient   dX = dY (theta . M)           App. "FLOP Calculation": backward = 2 x forward
//   weight gradient  dW = (dY^T X) . M             same passage
//   dense gradient   G  = dY^T X                   Algorithm 1, grad-growth step (|grad_theta L| on empty slots)
//   Mixed-Growing    prune / grow / rewrite        Algorithm 1
//
// Parity status: products pinned (brute force, dense-GEMM special case,
// adjoint identity); Mixed-Growing pinned (invariants, exhaustive tiny cases,
// independent re-implementation, SET/RigL special cases of Table 2).
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

extern "C" {

// ---------------------------------------------------------------- products
// Y[t,o] = sum_i M[o,i] * W[o,i] * X[t,i]
void mst_oracle_fwd(int64_t T, int64_t O, int64_t I, const double* X, const double* W, const uint8_t* M, double* Y) {
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < T; ++t)
    for (int64_t o = 0; o < O; ++o) {
      double s = 0.0;
      for (int64_t i = 0; i < I; ++i)
        if (M[o * I + i]) s += W[o * I + i] * X[t * I + i];
      Y[t * O + o] = s;
    }
}

// dX[t,i] = sum_o dY[t,o] * M[o,i] * W[o,i]
void mst_oracle_bwd_x(int64_t T, int64_t O, int64_t I, const double* dY, const double* W, const uint8_t* M, double* dX) {
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < T; ++t) {
    for (int64_t i = 0; i < I; ++i) dX[t * I + i] = 0.0;
    for (int64_t o = 0; o < O; ++o) {
      const double g = dY[t * O + o];
      for (int64_t i = 0; i < I; ++i)
        if (M[o * I + i]) dX[t * I + i] += g * W[o * I + i];
    }
  }
}

// dW[o,i] = M[o,i] * sum_t dY[t,o] * X[t,i]; entries off the mask are not computed and left exactly 0.
void mst_oracle_dw(int64_t T, int64_t O, int64_t I, const double* dY, const double* X, const uint8_t* M, double* dW) {
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t o = 0; o < O; ++o)
    for (int64_t i = 0; i < I; ++i) {
      if (!M[o * I + i]) { dW[o * I + i] = 0.0; continue; }
      double s = 0.0;
      for (int64_t t = 0; t < T; ++t) s += dY[t * O + o] * X[t * I + i];
      dW[o * I + i] = s;
    }
}

// G[o,i] = sum_t dY[t,o] * X[t,i] for every entry.
void mst_oracle_dense_grad(int64_t T, int64_t O, int64_t I, const double* dY, const double* X, double* G) {
#pragma omp parallel for schedule(static)
  for (int64_t o = 0; o < O; ++o)
    for (int64_t i = 0; i < I; ++i) {
      double s = 0.0;
      for (int64_t t = 0; t < T; ++t) s += dY[t * O + o] * X[t * I + i];
      G[o * I + i] = s;
    }
}

// The same sums evaluated only at listed output positions (full-size spot checks).
void mst_oracle_fwd_at(int64_t O, int64_t I, const double* X, const double* W, const uint8_t* M,
                       int64_t n, const int64_t* t_idx, const int64_t* o_idx, double* out) {
  (void)O;
#pragma omp parallel for schedule(static)
  for (int64_t s = 0; s < n; ++s) {
    const int64_t t = t_idx[s], o = o_idx[s];
    double a = 0.0;
    for (int64_t i = 0; i < I; ++i)
      if (M[o * I + i]) a += W[o * I + i] * X[t * I + i];
    out[s] = a;
  }
}

void mst_oracle_bwd_x_at(int64_t O, int64_t I, const double* dY, const double* W, const uint8_t* M,
                         int64_t n, const int64_t* t_idx, const int64_t* i_idx, double* out) {
#pragma omp parallel for schedule(static)
  for (int64_t s = 0; s < n; ++s) {
    const int64_t t = t_idx[s], i = i_idx[s];
    double a = 0.0;
    for (int64_t o = 0; o < O; ++o)
      if (M[o * I + i]) a += dY[t * O + o] * W[o * I + i];
    out[s] = a;
  }
}

// out[s] = sum_t dY[t,o_s] X[t,i_s]  (mask not applied: the caller picks the positions)
void mst_oracle_grad_at(int64_t T, int64_t O, int64_t I, const double* dY, const double* X,
                        int64_t n, const int64_t* o_idx, const int64_t* i_idx, double* out) {
#pragma omp parallel for schedule(static)
  for (int64_t s = 0; s < n; ++s) {
    const int64_t o = o_idx[s], i = i_idx[s];
    double a = 0.0;
    for (int64_t t = 0; t < T; ++t) a += dY[t * O + o] * X[t * I + i];
    out[s] = a;
  }
}

// ------------------------------------------------------ random-growth stream
// RandK of Algorithm 1 needs a generator; the paper names none.  Candidates are
// ranked by the outputs of SplitMix64 (Steele, Lea, Flood 2014): the key of flat
// index f is output number f+1 of a SplitMix64 generator whose state is derived
// from (seed, step, layer) by three chained first-outputs.
static inline uint64_t sm64_mix(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}
static const uint64_t SM64_GAMMA = 0x9E3779B97F4A7C15ULL;

uint64_t mst_oracle_stream(uint64_t seed, uint64_t step, int64_t layer_id) {
  uint64_t a = sm64_mix(seed + SM64_GAMMA);
  uint64_t b = sm64_mix((a ^ step) + SM64_GAMMA);
  return sm64_mix((b ^ (uint64_t)layer_id) + SM64_GAMMA);
}
uint64_t mst_oracle_rand_key(uint64_t stream, int64_t flat_index) {
  return sm64_mix(stream + SM64_GAMMA * (uint64_t)(flat_index + 1));
}

// ----------------------------------------------------------------- counts
// Algorithm 1, count lines, with the readings:
//   n_prune0 = floor(zeta * nnz)                      (no rounding is printed; floor, like the N_rand line)
//   n_grow   = n_prune + (n_target - nnz)             (sign chosen so that the layer reaches its target sparsity s_l')
//   n_prune clamped to [max(0, nnz - n_target), min(nnz, N - n_target)]  (so that 0 <= n_grow <= free slots)
//   n_rand   = floor(n_grow * R),  n_grad = n_grow - n_rand
// out = {n_prune, n_grow, n_rand, n_grad}.  Returns 0, or 2 when no feasible counts exist.
int mst_oracle_mg_counts(double zeta, int64_t nnz, int64_t n_target, int64_t N, double R, int64_t* out) {
  if (n_target < 0) n_target = nnz;
  if (n_target > N || nnz < 0 || nnz > N || !(zeta >= 0.0 && zeta <= 1.0) || !(R >= 0.0 && R <= 1.0)) return 2;
  int64_t n_prune = (int64_t)std::floor(zeta * (double)nnz);
  n_prune = std::max<int64_t>(n_prune, std::max<int64_t>(nnz - n_target, 0));
  n_prune = std::min<int64_t>(n_prune, std::min<int64_t>(nnz, N - n_target));
  const int64_t n_grow = n_prune - nnz + n_target;
  const int64_t n_rand = (int64_t)std::floor((double)n_grow * R);
  out[0] = n_prune; out[1] = n_grow; out[2] = n_rand; out[3] = n_grow - n_rand;
  return 0;
}

// ------------------------------------------------------------ Mixed-Growing
static inline uint32_t abs_bits(float v) {
  uint32_t u; std::memcpy(&u, &v, 4);
  return u & 0x7FFFFFFFu;
}

// One topology update of one layer (Algorithm 1), given the counts.
//   W [O*I] float32 in/out: stored weights (bf16 weights are passed widened); on exit W = W . M_new
//   M [O*I] in/out mask
//   G [O*I] float32 dense gradient (may be NULL when n_grad == 0)
//   I_prune / I_grad / I_rand: outputs (flat indices, selection order), may be NULL
// Orders (ties broken by the flat index o*I+i, smaller first):
//   prune: ascending |w| over active entries
//   grad : descending |g| over entries that were inactive before the update
//          (allow_regrow_pruned != 0: over inactive and just-pruned entries)
//   rand : ascending SplitMix64 key over entries inactive before the update and not picked by grad
// Returns 0 ok, 1 non-finite key met, 2 counts infeasible.
int mst_oracle_mg_update(int64_t O, int64_t I, float* W, uint8_t* M, const float* G,
                         int64_t n_prune, int64_t n_grad, int64_t n_rand,
                         uint64_t seed, uint64_t step, int64_t layer_id, int allow_regrow_pruned,
                         int64_t* I_prune, int64_t* I_grad, int64_t* I_rand, float prune_grad_weight) {
  const int64_t N = O * I;
  typedef std::pair<uint64_t, int64_t> KI;
  std::vector<uint8_t> old_mask(M, M + N);

  // prune: the n_prune active entries of smallest magnitude
  std::vector<KI> act;
  for (int64_t f = 0; f < N; ++f)
    if (old_mask[f]) {
      // prune key: |theta| (Mixed-Growing, SET, RigL) or |theta| + lambda |grad| (the MEST column of the scheme
      // table), the latter formed in float32 with one rounding per operation
      uint32_t k = abs_bits(W[f]);
      if (prune_grad_weight != 0.0f) {
        if (!G) return 2;
        volatile float prod = prune_grad_weight * std::fabs(G[f]);
        volatile float sum = std::fabs(W[f]) + prod;
        k = abs_bits(sum);
      }
      if (n_prune > 0 && k >= 0x7F800000u) return 1;   // keys are only examined when something is selected
      act.push_back(KI(k, f));
    }
  if (n_prune < 0 || n_prune > (int64_t)act.size() || n_grad < 0 || n_rand < 0) return 2;
  std::sort(act.begin(), act.end());
  std::vector<uint8_t> pruned(N, 0);
  for (int64_t j = 0; j < n_prune; ++j) {
    pruned[act[j].second] = 1;
    if (I_prune) I_prune[j] = act[j].second;
  }

  // gradient growth: the n_grad candidates of largest |g|
  std::vector<uint8_t> grown(N, 0);
  if (n_grad > 0) {
    if (!G) return 2;
    std::vector<KI> cand;
    for (int64_t f = 0; f < N; ++f)
      if (!old_mask[f] || (allow_regrow_pruned && pruned[f])) {
        const uint32_t k = abs_bits(G[f]);
        if (k >= 0x7F800000u) return 1;
        cand.push_back(KI((uint64_t)(0xFFFFFFFFu - k), f));   // descending |g|, then ascending index
      }
    if (n_grad > (int64_t)cand.size()) return 2;
    std::sort(cand.begin(), cand.end());
    for (int64_t j = 0; j < n_grad; ++j) {
      grown[cand[j].second] = 1;
      if (I_grad) I_grad[j] = cand[j].second;
    }
  }

  // random growth: n_rand of the remaining empty slots, ranked by the SplitMix64 key
  if (n_rand > 0) {
    const uint64_t stream = mst_oracle_stream(seed, step, layer_id);
    std::vector<KI> cand;
    for (int64_t f = 0; f < N; ++f)
      if (!old_mask[f] && !grown[f]) cand.push_back(KI(mst_oracle_rand_key(stream, f), f));
    if (n_rand > (int64_t)cand.size()) return 2;
    std::sort(cand.begin(), cand.end());
    for (int64_t j = 0; j < n_rand; ++j) {
      grown[cand[j].second] = 2;
      if (I_rand) I_rand[j] = cand[j].second;
    }
  }

  // mask rewrite, then theta <- theta . M.  Weights under the old mask were already zero
  // off-mask, so a grown entry starts at +0; an entry both pruned and regrown keeps its value.
  for (int64_t f = 0; f < N; ++f) {
    uint8_t m = old_mask[f];
    if (pruned[f]) m = 0;
    if (grown[f]) m = 1;
    M[f] = m;
    if (!m || !old_mask[f]) W[f] = 0.0f;
  }
  return 0;
}

}  // extern "C"
