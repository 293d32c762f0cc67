"""Sparsity-Variation schedule of Sec. 3.1 / 3.2 in plain Python (test infrastructure).

The printed equations for S_t put "100 %" where the dense model's sparsity belongs and wrap the whole ratio in the
floor; read as the cited cubic schedule s_t = s_f + (s_i - s_f)(1 - x)^3 with the stepwise x = floor(t'/Delta)/N they
give the N sparsity stages the text describes.  Parity unpinned: the paper prints no value of S_t or zeta_t, and its
219.4 G average-FLOPs figure is not reproducible from the text; the pins in the tests are closed forms of this reading.
"""
import math


def sparsity(step, S_M=0.96, N=5, delta_w=2000, t_ultra=100000, delta_r=2000):
    T_W, T_R = N * delta_w, N * delta_r
    if step < T_W:                                  # warm-up: dense -> S_M
        x = (step // delta_w) / N
        return S_M + (0.0 - S_M) * (1.0 - x) ** 3
    if step < T_W + t_ultra:                        # ultra-sparsification
        return S_M
    if step < T_W + t_ultra + T_R:                  # restoration: S_M -> dense
        x = ((step - T_W - t_ultra) // delta_r) / N
        return 0.0 + (S_M - 0.0) * (1.0 - x) ** 3
    return 0.0


def update_fraction(step, zeta1=0.3, decay=1.0, N=5, delta_w=2000, t_ultra=100000, delta_r=2000):
    # boundaries T_0 = 0, T_1 = T_W + T_U, T_2 = T_1 + Delta_R, ..., T_{N+1} = T_1 + T_R
    T = [0, N * delta_w + t_ultra]
    for _ in range(N):
        T.append(T[-1] + delta_r)
    for i in range(1, len(T)):
        if T[i - 1] <= step < T[i]:
            zeta_i = zeta1 * decay ** (i - 1)
            return zeta_i / 2.0 * (1.0 + math.cos((step - T[i - 1]) / (T[i] - T[i - 1]) * math.pi))
    return 0.0
