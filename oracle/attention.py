"""Strided sparse self-attention, the plain definition (fp64, CPU).

TEST INFRASTRUCTURE ONLY, like the rest of this package.

Sec. 3.3: output i is the softmax-weighted sum of the values at the positions S_i it attends to, with scores
(W_q x_i)(W_k x_j)^T / sqrt(d).  In the unfactorized strided pattern every head uses the same S_i: the previous
`stride` positions (i itself included) together with every `stride`-th earlier position.  The printed set formula
joins the two parts with an intersection sign; the text, the figure and the FLOP ratios of the appendix table
(22.03 % for stride 256, 12.07 % for stride 128 at n = 1024) fix the union, which is what is written here.

Pins (tests/test_oracle_attention.py): the mask's population against the printed ratios, the reduction to causal
softmax attention when stride >= n (computed there by a separate formula), constant values, a hand example, and a
position-by-position loop on small cases.  The backward pass (the derivative of that definition: softmax Jacobian
and the three matrix products) is pinned by central differences of the forward function, by the directional
identity <dO, dOut> = <dQ, dq> + <dK, dk> + <dV, dv>, and by a position-by-position loop.
"""
from __future__ import annotations

import numpy as np


def strided_mask(n: int, stride: int) -> np.ndarray:
    """bool [n, n]: entry (i, j) is True when position i attends to position j."""
    i = np.arange(n)[:, None]
    j = np.arange(n)[None, :]
    back = i - j
    return (back >= 0) & ((back < stride) | (back % stride == 0))


def strided_attention(Q, K, V, stride: int):
    """Q, K, V: [batch, heads, n, d].  Returns (out [batch, heads, n, d], lse [batch, heads, n]) in float64;
    lse is the log of the softmax denominator (natural log, scaled scores)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    n, d = Q.shape[-2], Q.shape[-1]
    keep = strided_mask(n, stride)
    s = np.matmul(Q, np.swapaxes(K, -1, -2)) / np.sqrt(float(d))
    s = np.where(keep, s, -np.inf)
    m = s.max(axis=-1, keepdims=True)
    e = np.exp(s - m)
    z = e.sum(axis=-1, keepdims=True)
    return np.matmul(e / z, V), (m + np.log(z))[..., 0]


def strided_attention_bwd(Q, K, V, dO, stride: int):
    """Gradients of strided_attention's output with respect to Q, K, V for the upstream gradient dO
    ([batch, heads, n, d] each, float64).  With P the masked softmax of the scaled scores:
    dV = P^T dO;  dP = dO V^T;  dS = P * (dP - rowsum(dP * P));  dQ = dS K / sqrt(d);  dK = dS^T Q / sqrt(d)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    dO = np.asarray(dO, dtype=np.float64)
    n, d = Q.shape[-2], Q.shape[-1]
    keep = strided_mask(n, stride)
    scale = 1.0 / np.sqrt(float(d))
    s = np.where(keep, np.matmul(Q, np.swapaxes(K, -1, -2)) * scale, -np.inf)
    e = np.exp(s - s.max(axis=-1, keepdims=True))
    P = e / e.sum(axis=-1, keepdims=True)
    dV = np.matmul(np.swapaxes(P, -1, -2), dO)
    dP = np.matmul(dO, np.swapaxes(V, -1, -2))
    dS = P * (dP - (dP * P).sum(axis=-1, keepdims=True))
    dQ = np.matmul(dS, K) * scale
    dK = np.matmul(np.swapaxes(dS, -1, -2), Q) * scale
    return dQ, dK, dV


def strided_attention_at(Q, K, V, stride: int, b, h, i):
    """Sampled outputs: rows (b[k], h[k], i[k]) of strided_attention, one position at a time."""
    Q = np.asarray(Q); K = np.asarray(K); V = np.asarray(V)
    d = Q.shape[-1]
    out = np.empty((len(b), d), dtype=np.float64)
    for k, (bb, hh, ii) in enumerate(zip(b, h, i)):
        js = [j for j in range(ii + 1) if ii - j < stride or (ii - j) % stride == 0]
        q = Q[bb, hh, ii].astype(np.float64)
        s = np.array([np.dot(q, K[bb, hh, j].astype(np.float64)) for j in js]) / np.sqrt(float(d))
        p = np.exp(s - s.max())
        p /= p.sum()
        out[k] = sum(pj * V[bb, hh, j].astype(np.float64) for pj, j in zip(p, js))
    return out
