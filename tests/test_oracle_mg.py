"""Pins for the oracle's Mixed-Growing update (Algorithm 1) and its counts (CPU only)."""
import itertools

import numpy as np
import pytest

import oracle


# ------------------------------------------------------------------ counts
def test_counts_follow_algorithm_lines():
    # zeta=0.3, nnz=589824, same target, R=0.25 (the paper's operating point)
    n_prune, n_grow, n_rand, n_grad = oracle.mg_counts(0.3, 589824, 589824, 2359296, 0.25)
    assert n_prune == 176947 and n_grow == 176947          # floor(0.3*589824)=floor(176947.2)
    assert n_rand == 44236 and n_grad == 132711            # floor(176947*0.25)=floor(44236.75)
    # target differs from current: grow - prune equals the change in active count
    n_prune, n_grow, n_rand, n_grad = oracle.mg_counts(0.1, 1000, 1200, 5000, 0.5)
    assert (n_prune, n_grow, n_rand, n_grad) == (100, 300, 150, 150)
    # warm-up style drop larger than zeta allows: prune count is raised to reach the target, nothing grows
    assert oracle.mg_counts(0.1, 1000, 400, 5000, 0.25) == (600, 0, 0, 0)
    # restoration to fully dense: prune count lowered so growth fits the free slots
    assert oracle.mg_counts(0.3, 1000, 5000, 5000, 0.25) == (0, 4000, 1000, 3000)
    # n_target < 0 keeps nnz
    assert oracle.mg_counts(0.5, 10, -1, 40, 0.0) == (5, 5, 0, 5)
    with pytest.raises(ValueError):
        oracle.mg_counts(0.3, 10, 50, 40, 0.25)


# ------------------------------------------------------- random-growth keys
def test_rand_keys_are_splitmix64_outputs():
    # Published SplitMix64 test vector: state 0 yields e220a8397b1dcdaf, 6e789e6aa1b965f4, 06c45d188009454f.
    L = oracle.lib()
    got = [int(L.mst_oracle_rand_key(0, f)) for f in range(3)]
    assert got == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    # stream derivation = three chained first outputs
    M64 = (1 << 64) - 1

    def mix(z):
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
        return z ^ (z >> 31)

    G = 0x9E3779B97F4A7C15
    seed, step, layer = 0x1234, 77, 5
    a = mix((seed + G) & M64); b = mix(((a ^ step) + G) & M64); c = mix(((b ^ layer) + G) & M64)
    assert int(L.mst_oracle_stream(seed, step, layer)) == c
    assert oracle.rand_key(seed, step, layer, 9) == mix((c + G * 10) & M64)


# ---------------------------------------------------- independent reference
def _abs_bits(a):
    return (np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) & 0x7FFFFFFF).astype(np.uint64)


def _mg_numpy(W, M, G, n_prune, n_grad, n_rand, seed, step, layer, allow=False):
    """Same rule written with numpy lexsort instead of sorting (key,index) pairs."""
    O, I = W.shape
    Wf, Mf = W.reshape(-1).copy(), M.reshape(-1).astype(bool).copy()
    idx = np.arange(O * I)
    act = idx[Mf]
    order = np.lexsort((act, _abs_bits(Wf[act])))
    I_prune = act[order[:n_prune]]
    cand_mask = ~Mf
    if allow:
        cand_mask = cand_mask.copy(); cand_mask[I_prune] = True
    cand = idx[cand_mask]
    I_grad = np.zeros(0, dtype=np.int64)
    if n_grad:
        gk = _abs_bits(G.reshape(-1)[cand])
        order = np.lexsort((cand, -gk.astype(np.int64)))
        I_grad = cand[order[:n_grad]]
    rc = np.setdiff1d(idx[~Mf], I_grad)
    keys = np.array([oracle.rand_key(seed, step, layer, int(f)) for f in rc], dtype=np.uint64)
    order = np.lexsort((rc, keys))
    I_rand = rc[order[:n_rand]]
    newM = Mf.copy(); newM[I_prune] = False; newM[I_grad] = True; newM[I_rand] = True
    newW = np.where(newM & Mf, Wf, np.float32(0)).astype(np.float32)
    return newW.reshape(O, I), newM.astype(np.uint8).reshape(O, I), I_prune, I_grad, I_rand


def _case(rng, O, I, density, ties=True):
    M = (rng.random((O, I)) < density).astype(np.uint8)
    W = (rng.standard_normal((O, I)) * 0.02).astype(np.float32)
    G = rng.standard_normal((O, I)).astype(np.float32)
    if ties:   # duplicated magnitudes, signed zeros, opposite signs
        W.reshape(-1)[::5] = np.float32(0.0)
        W.reshape(-1)[1::7] = np.float32(-0.0)
        W.reshape(-1)[2::9] = np.float32(0.01)
        W.reshape(-1)[3::11] = np.float32(-0.01)
        G.reshape(-1)[::4] = np.float32(0.5)
        G.reshape(-1)[1::6] = np.float32(-0.5)
    W = np.where(M == 1, W, np.float32(0.0)).astype(np.float32)      # off-mask weights are +0.0
    return W, M, G


@pytest.mark.parametrize("O,I,density,zeta,R,dn,allow", [
    (6, 8, 0.4, 0.3, 0.25, 0, False), (9, 13, 0.2, 0.5, 0.5, 7, False), (9, 13, 0.6, 0.2, 0.0, -20, False),
    (12, 32, 0.1, 0.1, 1.0, 0, False), (5, 5, 0.5, 1.0, 0.25, 3, False), (16, 48, 0.3, 0.3, 0.25, 0, True),
    (7, 40, 0.25, 0.0, 0.25, 0, False)])
def test_update_matches_independent_implementation(O, I, density, zeta, R, dn, allow):
    rng = np.random.default_rng(O * 1000 + I)
    W, M, G = _case(rng, O, I, density)
    nnz = int(M.sum())
    n_target = int(np.clip(nnz + dn, 0, O * I))
    n_prune, n_grow, n_rand, n_grad = oracle.mg_counts(zeta, nnz, n_target, O * I, R)
    Wn, Mn, ip, ig, ir = oracle.mg_update(W, M, G, n_prune, n_grad, n_rand, 99, 3, 2, allow)
    W2, M2, ip2, ig2, ir2 = _mg_numpy(W, M, G, n_prune, n_grad, n_rand, 99, 3, 2, allow)
    np.testing.assert_array_equal(Mn, M2)
    np.testing.assert_array_equal(Wn.view(np.uint32), W2.view(np.uint32))
    np.testing.assert_array_equal(ip, ip2); np.testing.assert_array_equal(ig, ig2); np.testing.assert_array_equal(ir, ir2)
    # invariants
    assert int(Mn.sum()) == n_target
    assert len(set(ip)) == n_prune and len(set(ig)) == n_grad and len(set(ir)) == n_rand
    Mf = M.reshape(-1).astype(bool)
    assert Mf[ip].all() and not Mf[ir].any() and not (set(ig) & set(ir))
    if not allow:
        assert not Mf[ig].any() and not (set(ip) & (set(ig) | set(ir)))    # a just-pruned slot is never regrown
    assert np.all(Wn.reshape(-1)[np.concatenate([ir, np.setdiff1d(ig, ip)])].view(np.uint32) == 0)   # grown = +0.0
    assert np.all(Wn[Mn == 0].view(np.uint32) == 0)


def test_selection_thresholds():
    rng = np.random.default_rng(5)
    W, M, G = _case(rng, 20, 30, 0.4, ties=False)
    nnz = int(M.sum())
    n_prune, _, n_rand, n_grad = oracle.mg_counts(0.3, nnz, nnz, 600, 0.25)
    Wn, Mn, ip, ig, ir = oracle.mg_update(W, M, G, n_prune, n_grad, n_rand, 1, 2, 3)
    a = np.abs(W.reshape(-1)); g = np.abs(G.reshape(-1))
    surv = np.setdiff1d(np.nonzero(M.reshape(-1))[0], ip)
    assert a[ip].max() <= a[surv].min()
    not_grown = np.setdiff1d(np.nonzero(M.reshape(-1) == 0)[0], ig)
    assert g[ig].min() >= g[not_grown].max()


def test_exhaustive_tiny_layers():
    # Brute force over all subsets: the pruned set minimises, the grown set maximises, the order-statistic sums,
    # and under the index tie-break both are the lexicographically first such subsets.
    rng = np.random.default_rng(21)
    for trial in range(6):
        O, I = 3, 4
        M = (rng.random((O, I)) < 0.5).astype(np.uint8)
        if M.sum() < 3 or M.sum() > 9:
            continue
        W = rng.integers(-2, 3, size=(O, I)).astype(np.float32) * M      # many ties
        G = rng.integers(-2, 3, size=(O, I)).astype(np.float32)
        act = list(np.nonzero(M.reshape(-1))[0]); ina = list(np.nonzero(M.reshape(-1) == 0)[0])
        n_prune, n_grad = 2, 2
        _, _, ip, ig, _ = oracle.mg_update(W, M, G, n_prune, n_grad, 0, 0, 0, 0)
        aw, ag = np.abs(W.reshape(-1)), np.abs(G.reshape(-1))
        best_p = min(itertools.combinations(act, n_prune), key=lambda s: (sum(aw[list(s)]), s))
        best_g = min(itertools.combinations(ina, n_grad), key=lambda s: (-sum(ag[list(s)]), s))
        assert sorted(ip) == list(best_p) and sorted(ig) == list(best_g)


def test_special_cases_of_the_scheme_table():
    rng = np.random.default_rng(31)
    W, M, G = _case(rng, 10, 24, 0.3)
    nnz = int(M.sum())
    # R = 0: RigL (all growth by gradient magnitude); R = 1: SET (all growth random)
    c0 = oracle.mg_counts(0.3, nnz, nnz, 240, 0.0); c1 = oracle.mg_counts(0.3, nnz, nnz, 240, 1.0)
    assert c0[2] == 0 and c0[3] == c0[1] and c1[3] == 0 and c1[2] == c1[1]
    _, M0, ip0, ig0, ir0 = oracle.mg_update(W, M, G, c0[0], c0[3], c0[2], 1, 1, 1)
    _, M1, ip1, ig1, ir1 = oracle.mg_update(W, M, None, c1[0], c1[3], c1[2], 1, 1, 1)
    assert len(ir0) == 0 and len(ig1) == 0 and int(M0.sum()) == int(M1.sum()) == nnz
    np.testing.assert_array_equal(ip0, ip1)                   # same magnitude pruning in both
    # zeta = 0, same target: identity
    Wn, Mn, *_ = oracle.mg_update(W, M, G, 0, 0, 0, 1, 1, 1)
    np.testing.assert_array_equal(Mn, M); np.testing.assert_array_equal(Wn.view(np.uint32), W.view(np.uint32))
    # target = N: all-ones mask; target = 0: empty
    c = oracle.mg_counts(0.3, nnz, 240, 240, 0.25)
    _, Mn, *_ = oracle.mg_update(W, M, G, c[0], c[3], c[2], 1, 1, 1)
    assert Mn.all()
    c = oracle.mg_counts(0.3, nnz, 0, 240, 0.25)
    Wn, Mn, *_ = oracle.mg_update(W, M, G, c[0], c[3], c[2], 1, 1, 1)
    assert not Mn.any() and not Wn.any()


def test_signed_zero_and_sign_do_not_affect_order():
    W = np.array([[-0.0, 0.5, -0.25, 0.25, 0.0]], dtype=np.float32)
    M = np.ones((1, 5), dtype=np.uint8)
    _, _, ip, _, _ = oracle.mg_update(W, M, None, 4, 0, 0, 0, 0, 0)
    assert list(ip) == [0, 4, 2, 3]          # |.| order, ties by index: -0.0 (idx 0) before +0.0 (idx 4); -.25 before +.25


def test_nonfinite_keys_are_rejected():
    W = np.array([[1.0, np.inf, 2.0]], dtype=np.float32); M = np.ones((1, 3), dtype=np.uint8)
    with pytest.raises(oracle.NonFinite):
        oracle.mg_update(W, M, None, 1, 0, 0, 0, 0, 0)
    W = np.array([[1.0, 0.0, 2.0]], dtype=np.float32); M = np.array([[1, 0, 1]], dtype=np.uint8)
    G = np.array([[0.0, np.nan, 0.0]], dtype=np.float32)
    with pytest.raises(oracle.NonFinite):
        oracle.mg_update(W, M, G, 1, 1, 0, 0, 0, 0)


def test_random_growth_is_uniform_over_positions():
    # chi-square of how often each empty slot is picked over many (seed, step) streams
    O, I = 4, 16
    M = np.zeros((O, I), dtype=np.uint8); M[:, ::4] = 1
    W = np.ones((O, I), dtype=np.float32) * M
    empty = np.nonzero(M.reshape(-1) == 0)[0]
    hits = np.zeros(O * I)
    trials, k = 600, 12
    for s in range(trials):
        _, _, _, _, ir = oracle.mg_update(W, M, None, 0, 0, k, 1000 + s, s % 7, 3)
        hits[ir] += 1
    assert hits[M.reshape(-1) == 1].sum() == 0
    expect = trials * k / len(empty)
    chi2 = ((hits[empty] - expect) ** 2 / expect).sum()
    assert chi2 < 85.0        # 47 dof: mean 47, the 99.9th percentile is about 82
    # different steps give different picks, same (seed, step, layer) repeats exactly
    a = oracle.mg_update(W, M, None, 0, 0, k, 5, 1, 3)[4]; b = oracle.mg_update(W, M, None, 0, 0, k, 5, 2, 3)[4]
    c = oracle.mg_update(W, M, None, 0, 0, k, 5, 1, 3)[4]
    assert list(a) == list(c) and list(a) != list(b)


def test_to_csr_roundtrip():
    rng = np.random.default_rng(41)
    W, M, _ = _case(rng, 9, 17, 0.3)
    rp, ci, v = oracle.to_csr(W, M)
    D = np.zeros_like(W); Mb = np.zeros_like(M)
    for o in range(9):
        cols = ci[rp[o]:rp[o + 1]]
        assert np.all(np.diff(cols) > 0)
        D[o, cols] = v[rp[o]:rp[o + 1]]; Mb[o, cols] = 1
    np.testing.assert_array_equal(Mb, M); np.testing.assert_array_equal(D, W)
    np.testing.assert_array_equal(rp, np.concatenate([[0], np.cumsum(M.sum(1))]))


def test_mest_prune_key():
    # Scheme table, MEST column: prune by min(|theta| + lambda |grad|).  Independent float32 reference with numpy.
    rng = np.random.default_rng(61)
    W, M, G = _case(rng, 14, 40, 0.4)
    nnz = int(M.sum())
    lam = np.float32(0.37)
    n_prune = nnz // 3
    _, Mn, ip, _, _ = oracle.mg_update(W, M, G, n_prune, 0, 0, 0, 0, 0, False, float(lam))
    act = np.nonzero(M.reshape(-1))[0]
    key = (np.abs(W.reshape(-1)[act]).astype(np.float32) + (lam * np.abs(G.reshape(-1)[act]).astype(np.float32)).astype(np.float32)).astype(np.float32)
    order = np.lexsort((act, key.view(np.uint32)))
    np.testing.assert_array_equal(ip, act[order[:n_prune]])
    # lambda = 0 is the magnitude rule; a huge lambda orders by |grad|
    _, _, ip0, _, _ = oracle.mg_update(W, M, G, n_prune, 0, 0, 0, 0, 0, False, 0.0)
    _, _, ipm, _, _ = oracle.mg_update(W, M, None, n_prune, 0, 0, 0, 0, 0)
    np.testing.assert_array_equal(ip0, ipm)
    _, _, ipl, _, _ = oracle.mg_update(W, M, G, n_prune, 0, 0, 0, 0, 0, False, 1e6)
    g = np.abs(G.reshape(-1))
    surv = np.setdiff1d(act, ipl)
    assert g[ipl].max() <= g[surv].min() + 1e-6
    with pytest.raises(ValueError):
        oracle.mg_update(W, M, None, n_prune, 0, 0, 0, 0, 0, False, 0.5)      # the criterion needs the gradient
