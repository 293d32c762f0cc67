"""A whole Sparsity-Variation trajectory on one small transformer block (needs a GPU).

Dense start -> warm-up stages -> ultra-sparse steps -> restoration stages -> dense again, driven by the host schedule
(S_t, zeta_t, Erdos-Renyi split) through mst_topology_update; after every update the layer's structure and values are
compared bit-exactly with the oracle's Algorithm 1 run from the same state, and the layer stays in one allocation.
"""
import numpy as np
import pytest

import mst_inputs
import oracle
import oracle.sv_schedule as ref

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2408_11746_b200 as mst
    from gpu_util import dev, export_csr, host, make_layer, rel_err, to_dev, value_bits, TOL


def test_dense_to_ultra_sparse_and_back():
    d_model, T = 64, 96
    shapes = [(o, i) for _, o, i in mst_inputs.block_shapes(d_model)]
    sc = mst.SvSchedule(0.96, 5, 2, 6, 2)                  # 5 stages of 2 steps, 6 ultra-sparse steps
    probs, layers, W, M = [], [], [], []
    for lid, (O, I) in enumerate(shapes):
        p = mst_inputs.uniform_layer("l%d" % lid, lid, O, I, T, "bf16", 1.0, 900 + lid)     # all-ones mask
        probs.append(p)
        layers.append(make_layer(p))                        # capacity O*I: restoration never reallocates
        W.append(p.W.copy()); M.append(p.mask.copy())
    rng = np.random.default_rng(9)
    total_steps = 5 * 2 + 6 + 5 * 2 + 1
    seen = []
    for t in range(1, total_steps + 1):
        S = mst.mst_sv_sparsity(sc, t)
        assert S == pytest.approx(ref.sparsity(t, 0.96, 5, 2, 6, 2), abs=1e-12)
        zeta = mst.mst_sv_update_fraction(sc, t, 0.3, 0.5)
        dens = mst.mst_er_densities(shapes, 1.0 - S)
        for lid, (O, I) in enumerate(shapes):
            p, L = probs[lid], layers[lid]
            target = int(round(dens[lid] * O * I))
            G = rng.standard_normal((O, I)).astype(np.float32)
            st = mst.mst_topology_update(L.handle, zeta, target, 0.25, 77, t, False, torch.from_numpy(G).to(dev()))
            c = oracle.mg_counts(zeta, int(M[lid].sum()), target, O * I, 0.25)
            assert (st.n_prune, st.n_rand, st.n_grad) == (c[0], c[2], c[3])
            W[lid], M[lid], *_ = oracle.mg_update(W[lid], M[lid], G, c[0], c[3], c[2], 77, t, lid)
            assert st.nnz_after == target == int(M[lid].sum())
            rp, ci, vb = export_csr(L, "bf16")
            rp_r, ci_r, v_r = oracle.to_csr(W[lid], M[lid])
            np.testing.assert_array_equal(rp, rp_r)
            np.testing.assert_array_equal(ci, ci_r)
            np.testing.assert_array_equal(vb, value_bits(v_r, "bf16"))
        seen.append(sum(int(m.sum()) for m in M) / sum(o * i for o, i in shapes))
    # dense -> about 4 % -> dense
    assert min(seen) == pytest.approx(0.04, abs=0.01) and seen[-1] == 1.0
    for lid, L in enumerate(layers):
        assert M[lid].all()
        L.validate()
        # the products still work on the restored (dense, mostly zero-valued) layer
        p = probs[lid]
        X = to_dev(p, "X")
        Y = torch.empty((T, p.out_features), dtype=torch.bfloat16, device=dev())
        L.fwd(X, Y, T)
        torch.cuda.synchronize()
        assert rel_err(host(Y), oracle.fwd(p.X, W[lid], M[lid])) <= TOL["bf16"]
        L.close()
