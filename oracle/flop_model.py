"""FLOP accounting of the paper's appendix "FLOP Calculation" (test infrastructure).

Used to pin the meaning of "useful FLOPs" of a sparse fully-connected layer
(Eq. (3): (1-S)(2I-1)O per token) against the totals the paper prints in its
performance table, and to check the strided-attention ratio of its attention
table.  Plain Python, exact integer/fraction arithmetic where possible.
"""
from __future__ import annotations


def fc_forward_flops(sparsity: float, in_features: int, out_features: int) -> float:
    """Eq. (3), one token: (1 - S)(2 I - 1) O."""
    return (1.0 - sparsity) * (2 * in_features - 1) * out_features


def training_flops(n_layers: int, n_embd: int, seq_len: int = 1024, vocab: int = 50304, sparsity: float = 0.0,
                   q_atten: float = 1.0) -> float:
    """Total training FLOPs per sequence (forward + backward = 3 x forward), appendix formulas.

    The value-reduction term is taken as Q * 2 * L * L * N_embd (the printed
    formula carries a stray factor; only this form reproduces the table).
    """
    L, d, ffw = seq_len, n_embd, 4 * n_embd
    kqv = L * fc_forward_flops(sparsity, d, 3 * d)
    scores = q_atten * 2 * L * L * d
    reduce_ = q_atten * 2 * L * L * d
    proj = L * fc_forward_flops(sparsity, d, d)
    ffw1 = L * fc_forward_flops(sparsity, d, ffw)
    ffw2 = L * fc_forward_flops(sparsity, ffw, d)
    transformer = n_layers * (kqv + scores + reduce_ + proj + ffw1 + ffw2)
    lm = L * fc_forward_flops(sparsity, d, vocab)
    return 3.0 * (transformer + lm)


def q_atten_strided(n: int, stride: int) -> float:
    """Fraction of the n x n score matrix kept when position i attends to its previous
    `stride` positions (itself included) and to every `stride`-th earlier position."""
    kept = 0
    for i in range(n):
        for j in range(i + 1):
            if i - j < stride or (i - j) % stride == 0:
                kept += 1
    return kept / float(n * n)


def erdos_renyi_densities(shapes, global_density: float):
    """Erdos-Renyi split (SET, cited by Sec. 3.2): d_l = eps (I_l + O_l) / (I_l O_l), eps set so the
    total number of active weights matches; layers that would exceed 1 are made dense and eps re-solved."""
    shapes = list(shapes)
    total = sum(o * i for o, i in shapes)
    want = global_density * total
    dense = [False] * len(shapes)
    while True:
        fixed = sum(o * i for (o, i), dn in zip(shapes, dense) if dn)
        denom = sum(o + i for (o, i), dn in zip(shapes, dense) if not dn)
        eps = (want - fixed) / denom
        d = [1.0 if dn else eps * (o + i) / (o * i) for (o, i), dn in zip(shapes, dense)]
        over = [(not dn) and dl > 1.0 for dl, dn in zip(d, dense)]
        if not any(over):
            return d, eps
        dense = [dn or ov for dn, ov in zip(dense, over)]
