"""The fidelity metrics of Section 4.2 (cosine, KL, Spearman, top-5) against scipy / closed forms, and
the qualitative behaviour the paper reports on synthetic keys (rank correlation high, exact case = 1)."""
import numpy as np
import scipy.stats

import oracle
from oracle import fidelity
from paper_2601_10155_b200 import synth


def test_metrics_match_scipy_and_closed_forms():
    rng = np.random.default_rng(0)
    a = rng.standard_normal((3, 4, 50))
    b = a + 0.3 * rng.standard_normal((3, 4, 50))
    b[..., 7] = b[..., 8]                                        # ties get average ranks
    rho = fidelity.spearman_rho(a, b)
    for i in range(3):
        for j in range(4):
            assert abs(rho[i, j] - scipy.stats.spearmanr(a[i, j], b[i, j]).statistic) < 1e-12
    p = scipy.special.softmax(a, axis=-1)
    qd = scipy.special.softmax(b, axis=-1)
    kl = fidelity.kl_divergence(p, qd)
    ref = scipy.stats.entropy(p, qd, axis=-1)
    np.testing.assert_allclose(kl, ref, rtol=1e-12)
    assert np.all(fidelity.kl_divergence(p, p) == 0)
    y = rng.standard_normal((5, 8))
    np.testing.assert_allclose(fidelity.cosine_similarity(y, 3.0 * y), 1.0, rtol=1e-12)
    np.testing.assert_allclose(fidelity.cosine_similarity(y, -y), -1.0, rtol=1e-12)
    w = np.array([[0.4, 0.3, 0.1, 0.05, 0.05, 0.04, 0.03, 0.03]])
    shuffled = w[:, [0, 1, 2, 7, 6, 5, 4, 3]]                    # top-5 of the permuted row shares 3 indices
    assert fidelity.topk_overlap(w, w, 5)[0] == 1.0
    assert fidelity.topk_overlap(w, shuffled, 5)[0] == 3 / 5


def test_exact_case_scores_perfectly_and_compressed_case_keeps_the_ranking():
    # N <= K: every key is a centroid, LOOKAT is exact attention
    w = synth.small_workload(B=1, n_q_heads=4, n_kv_heads=4, d_k=64, d_v=64, L=128, m=4, K=256, rank=16)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, 0.3)
    r = fidelity.evaluate(keys, v, q, m=4, iters=2)
    assert r["cosine"][0] > 1 - 1e-12 and r["spearman"][0] > 1 - 1e-12 and r["top5"][0] == 1.0
    assert r["kl"][0] < 1e-12 and r["compression"] == 32
    # real compression: 1024 keys on 256 centroids per subspace; ranking survives (rho around 0.95
    # on these keys), and more subspaces rank better than fewer
    w = synth.small_workload(B=2, n_q_heads=4, n_kv_heads=4, d_k=64, d_v=64, L=1024, m=4, K=256, rank=16)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, 0.1)
    calib = synth.make_calibration_keys(w, 2048)
    r2 = fidelity.evaluate(keys, v, q, m=2, iters=8, calib=calib)
    r8 = fidelity.evaluate(keys, v, q, m=8, iters=8, calib=calib)
    assert r2["spearman"][0] > 0.85 and r8["spearman"][0] > r2["spearman"][0]
    assert r8["cosine"][0] > 0.9 and r8["kl"][0] < r2["kl"][0]
