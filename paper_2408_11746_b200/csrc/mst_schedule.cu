// Host-side Sparsity-Variation driver (Sec. 3.1, Sec. 3.2): the global sparsity S_t over warm-up / ultra-sparse /
// restoration, the piecewise decaying cosine update fraction zeta_t, and the Erdos-Renyi split of a global density
// into per-layer densities.  Scalar code, no device work.
//
// Readings (the printed equations do not evaluate to a usable schedule as typeset):
//   * both phase equations are the cited cubic schedule s_t = s_f + (s_i - s_f)(1 - x)^3 (Zhu & Gupta), stepwise in
//     x = floor(t' / Delta) / N: warm-up from s_i = 0 to s_f = S_M, restoration from s_i = S_M to s_f = 0;
//   * zeta_t restarts at every restoration stage; the magnitudes zeta_i for i > 1 are not given in the paper: a geometric
//     decay zeta_i = zeta_1 * decay^(i-1) is offered ("Decay N-cosine"), decay = 1 gives "N-cosine".
#include <cmath>
#include <vector>

#include "mst.h"

extern "C" mst_status_t mst_sv_sparsity(const mst_sv_schedule_t* sc, int64_t step, double* sparsity) {
  if (!sc || !sparsity || step < 0) return MST_ERR_INVALID_ARG;
  if (!(sc->max_sparsity >= 0.0 && sc->max_sparsity <= 1.0) || sc->n_stages < 1 || sc->delta_w < 1 || sc->delta_r < 1 ||
      sc->t_ultra < 0)
    return MST_ERR_INVALID_ARG;
  const int64_t N = sc->n_stages, TW = N * sc->delta_w, TU = sc->t_ultra, TR = N * sc->delta_r;
  const double SM = sc->max_sparsity;
  double s;
  if (step < TW) {
    const double x = (double)(step / sc->delta_w) / (double)N;
    s = SM * (1.0 - (1.0 - x) * (1.0 - x) * (1.0 - x));
  } else if (step < TW + TU) {
    s = SM;
  } else if (step < TW + TU + TR) {
    const double x = (double)((step - TW - TU) / sc->delta_r) / (double)N;
    s = SM * (1.0 - x) * (1.0 - x) * (1.0 - x);
  } else {
    s = 0.0;
  }
  *sparsity = s;
  return MST_OK;
}

extern "C" mst_status_t mst_sv_update_fraction(const mst_sv_schedule_t* sc, int64_t step, double zeta1, double decay,
                                               double* zeta) {
  if (!sc || !zeta || step < 0 || !(zeta1 >= 0.0 && zeta1 <= 1.0) || !(decay >= 0.0 && decay <= 1.0)) return MST_ERR_INVALID_ARG;
  if (sc->n_stages < 1 || sc->delta_w < 1 || sc->delta_r < 1 || sc->t_ultra < 0) return MST_ERR_INVALID_ARG;
  const int64_t N = sc->n_stages, T1 = N * sc->delta_w + sc->t_ultra, TR = N * sc->delta_r;
  int64_t a, b;
  double mag = zeta1;
  if (step < T1) {
    a = 0;
    b = T1;
  } else if (step < T1 + TR) {
    const int64_t i = (step - T1) / sc->delta_r;  // restoration stage 0..N-1 -> interval i+2
    a = T1 + i * sc->delta_r;
    b = a + sc->delta_r;
    mag = zeta1 * std::pow(decay, (double)(i + 1));
  } else {
    *zeta = 0.0;
    return MST_OK;
  }
  const double pi = 3.14159265358979323846;
  *zeta = 0.5 * mag * (1.0 + std::cos((double)(step - a) / (double)(b - a) * pi));
  return MST_OK;
}

extern "C" mst_status_t mst_er_densities(int32_t n_layers, const int32_t* O, const int32_t* I, double global_density,
                                         double* densities) {
  if (n_layers < 1 || !O || !I || !densities || !(global_density >= 0.0 && global_density <= 1.0)) return MST_ERR_INVALID_ARG;
  double total = 0.0;
  for (int l = 0; l < n_layers; ++l) {
    if (O[l] < 1 || I[l] < 1) return MST_ERR_SHAPE;
    total += (double)O[l] * I[l];
  }
  const double want = global_density * total;
  std::vector<char> dense(n_layers, 0);
  for (int it = 0; it <= n_layers; ++it) {
    double fixed = 0.0, denom = 0.0;
    for (int l = 0; l < n_layers; ++l) {
      if (dense[l]) fixed += (double)O[l] * I[l];
      else denom += (double)O[l] + I[l];
    }
    const double eps = denom > 0.0 ? (want - fixed) / denom : 0.0;
    bool again = false;
    for (int l = 0; l < n_layers; ++l) {
      if (dense[l]) { densities[l] = 1.0; continue; }
      densities[l] = eps * ((double)O[l] + I[l]) / ((double)O[l] * I[l]);
      if (densities[l] > 1.0) { dense[l] = 1; again = true; }
    }
    if (!again) break;
  }
  for (int l = 0; l < n_layers; ++l) {
    if (densities[l] > 1.0) densities[l] = 1.0;
    if (densities[l] < 0.0) densities[l] = 0.0;
  }
  return MST_OK;
}
