"""Pins for the oracle's K-means update (Sec. 3.1, second approach: K-means directly in the document
embedding space; Sec. 4: the cluster centroid is the topic embedding).  One Lloyd iteration is the cosine
router (pinned in test_oracle_router.py) followed by this update."""
import numpy as np
from sklearn.cluster import KMeans

import moin_inputs as mi
import oracle


def _unit(a):
    return a / np.linalg.norm(a, axis=1, keepdims=True)


def _objective(x, c, assign):
    """Sum over the points of cos(x_i, c_assign(i)): what spherical K-means ascends."""
    ca = c[assign]
    return float(((x * ca).sum(1) / (np.linalg.norm(x, axis=1) * np.linalg.norm(ca, axis=1))).sum())


def test_update_is_the_member_mean_brute_force():
    rng = np.random.default_rng(0)
    x = rng.normal(size=(37, 5))
    assign = rng.integers(0, 6, size=37)
    old = rng.normal(size=(6, 5))
    out = oracle.kmeans_update(x, old, assign)
    for k in range(6):
        rows = [x[i] for i in range(37) if assign[i] == k]
        assert out["counts"][k] == len(rows)
        want = old[k] if not rows else [sum(r[d] for r in rows) / len(rows) for d in range(5)]
        np.testing.assert_allclose(out["centroids"][k], want, rtol=0, atol=1e-14)


def test_update_against_a_scatter_add_formulation():
    rng = np.random.default_rng(1)
    x = rng.normal(size=(5000, 48))
    assign = rng.integers(0, 300, size=5000)
    out = oracle.kmeans_update(x, np.zeros((300, 48)), assign)
    sums = np.zeros((300, 48))
    np.add.at(sums, assign, x)
    cnt = np.bincount(assign, minlength=300)
    np.testing.assert_allclose(out["centroids"][cnt > 0], sums[cnt > 0] / cnt[cnt > 0, None], atol=1e-12)
    assert np.array_equal(out["counts"], cnt)


def test_empty_cluster_keeps_its_centroid_and_bad_ids_are_ignored():
    x = np.array([[1.0, 0.0], [3.0, 0.0], [0.0, 5.0], [9.0, 9.0]])
    old = np.array([[7.0, 7.0], [8.0, 8.0], [6.0, 6.0]])
    out = oracle.kmeans_update(x, old, np.array([0, 0, 2, -1]))
    np.testing.assert_array_equal(out["centroids"], [[2.0, 0.0], [8.0, 8.0], [0.0, 5.0]])
    assert list(out["counts"]) == [2, 0, 1]


def test_point_order_does_not_matter_and_bf16_inputs_widen_exactly():
    rng = np.random.default_rng(2)
    xt, ot = mi.normal_bf16((600, 32), 1.0, 5, 1), mi.normal_bf16((20, 32), 1.0, 5, 2)
    xb, ob = mi.bf16_bits(xt), mi.bf16_bits(ot)
    assign = rng.integers(0, 20, size=600)
    a = oracle.kmeans_update(xb, ob, assign)
    perm = rng.permutation(600)
    b = oracle.kmeans_update(xb[perm], ob, assign[perm])
    np.testing.assert_allclose(a["centroids"], b["centroids"], atol=1e-13)
    c = oracle.kmeans_update(mi.bf16_to_f64(xt), mi.bf16_to_f64(ot), assign)   # same values as doubles
    np.testing.assert_array_equal(a["centroids"], c["centroids"])


def test_one_lloyd_iteration_equals_scikit_learn_on_unit_vectors():
    # For unit-norm points AND unit-norm centroids the Euclidean and the cosine nearest centroid coincide,
    # so one iteration of a textbook Lloyd K-means from the same start must give the same means.
    rng = np.random.default_rng(3)
    x = _unit(rng.normal(size=(2000, 16)))
    c0 = _unit(x[rng.choice(2000, size=25, replace=False)] + 0.05 * rng.normal(size=(25, 16)))
    assign = oracle.route(x, c0)["centroid"]
    mine = oracle.kmeans_update(x, c0, assign)["centroids"]
    km = KMeans(n_clusters=25, init=c0, n_init=1, max_iter=1, algorithm="lloyd", tol=0.0).fit(x)
    np.testing.assert_allclose(mine, km.cluster_centers_, atol=1e-10)


def test_lloyd_iterations_ascend_the_cosine_objective_and_recover_planted_clusters():
    # unit-norm points: the mean direction of a cluster maximises its members' summed cosine, and the router
    # re-assignment cannot lower it either, so the objective never decreases
    rc = mi.planted_router(K=40, Q=4000, D=32, seed=9, noise=0.3)
    x = mi.bf16_to_f64(rc.queries)
    planted = mi.bf16_to_f64(rc.centroids)
    rng = np.random.default_rng(4)
    c = planted + 0.4 * rng.normal(size=planted.shape) / np.sqrt(32)   # a perturbed start
    last = -np.inf
    for _ in range(6):
        assign = oracle.route(x, c)["centroid"]
        obj = _objective(x, c, assign)
        assert obj >= last - 1e-9
        last = obj
        c = oracle.kmeans_update(x, c, assign)["centroids"]
    cos = (_unit(c) * _unit(planted)).sum(1)
    assert cos.min() > 0.99
    assert (oracle.route(x, c)["centroid"] == rc.labels.numpy()).mean() > 0.999
