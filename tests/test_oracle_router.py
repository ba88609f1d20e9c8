"""Pins for the oracle's router (Sec. 3.3: nearest-neighbour search of the query embedding
over the topic embeddings; cosine similarity as the metric, lowest index on ties)."""
import numpy as np

import moin_inputs as mi
import oracle


def _unit(a):
    return a / np.linalg.norm(a, axis=1, keepdims=True)


def test_queries_equal_to_centroids_route_to_themselves():
    c = np.random.default_rng(0).normal(size=(40, 24))
    out = oracle.route(c * 3.0, c)   # self-cosine is 1 (Cauchy-Schwarz), scale-free
    assert np.array_equal(out["centroid"], np.arange(40))
    np.testing.assert_allclose(out["best"], 1.0, atol=1e-12)


def test_cosine_argmax_is_l2_argmin_for_unit_vectors():
    # |q - c|^2 = 2 - 2 cos for unit vectors: brute-force L2 nearest neighbour must agree.
    rng = np.random.default_rng(1)
    c, q = _unit(rng.normal(size=(64, 16))), _unit(rng.normal(size=(200, 16)))
    out = oracle.route(q, c)
    d2 = ((q[:, None, :] - c[None, :, :]) ** 2).sum(-1)
    assert np.array_equal(out["centroid"], d2.argmin(1))
    np.testing.assert_allclose(out["best"], 1.0 - 0.5 * d2.min(1), atol=1e-12)


def test_cosine_not_dot_product():
    # a long centroid with a smaller angle must lose to... nothing: cosine ignores length.
    c = np.array([[10.0, 10.0], [0.0, 1.0]])
    q = np.array([[0.1, 1.0]])
    out = oracle.route(q, c)
    assert out["centroid"][0] == 1          # dot product would pick 0
    np.testing.assert_allclose(out["best"][0], 1.0 / np.hypot(0.1, 1.0), atol=1e-12)


def test_positive_rescaling_changes_nothing():
    rng = np.random.default_rng(2)
    c, q = rng.normal(size=(30, 12)), rng.normal(size=(50, 12))
    a = oracle.route(q, c)
    b = oracle.route(q * rng.uniform(0.1, 9.0, size=(50, 1)), c * rng.uniform(0.1, 9.0, size=(30, 1)))
    assert np.array_equal(a["centroid"], b["centroid"])
    np.testing.assert_allclose(a["best"], b["best"], atol=1e-12)
    np.testing.assert_allclose(a["margin"], b["margin"], atol=1e-12)


def test_centroid_permutation_and_duplicates():
    rng = np.random.default_rng(3)
    c, q = rng.normal(size=(20, 8)), rng.normal(size=(64, 8))
    a = oracle.route(q, c)
    p = rng.permutation(20)
    b = oracle.route(q, c[p])
    assert np.array_equal(p[b["centroid"]], a["centroid"])
    # duplicate every centroid behind the originals: the lower index wins, margin is 0
    d = oracle.route(q, np.concatenate([c, c]))
    assert np.array_equal(d["centroid"], a["centroid"])
    np.testing.assert_allclose(d["margin"], 0.0, atol=0)


def test_margin_and_best_against_numpy_sort():
    rng = np.random.default_rng(4)
    c, q = rng.normal(size=(33, 10)), rng.normal(size=(41, 10))
    out = oracle.route(q, c)
    sim = _unit(q) @ _unit(c).T
    s = np.sort(sim, axis=1)
    np.testing.assert_allclose(out["best"], s[:, -1], atol=1e-12)
    np.testing.assert_allclose(out["margin"], s[:, -1] - s[:, -2], atol=1e-12)


def test_centroid_to_expert_map_and_retained_rows():
    # "MoIN-5k": routed topic may have no adapter (-1); "MoIN-4697": router over retained rows only.
    rng = np.random.default_rng(5)
    c, q = rng.normal(size=(12, 6)), rng.normal(size=(30, 6))
    cmap = np.arange(12, dtype=np.int32)
    cmap[[2, 7]] = -1
    full = oracle.route(q, c, cmap)
    assert np.array_equal(full["expert"], cmap[full["centroid"]])
    kept = np.array([k for k in range(12) if k not in (2, 7)])
    sub = oracle.route(q, c[kept], kept.astype(np.int32))
    sim = _unit(q) @ _unit(c).T
    sim[:, [2, 7]] = -np.inf
    assert np.array_equal(sub["expert"], sim.argmax(1))


def test_degenerate_vectors():
    c = np.array([[0.0, 0.0], [1.0, 0.0], [0.0, 1.0]])
    out = oracle.route(np.array([[1.0, 0.1], [0.0, 0.0], [-1.0, -1.0]]), c)
    assert out["centroid"][0] == 1           # zero-norm centroid never chosen
    assert out["centroid"][1] == 0           # zero-norm query: id 0
    assert out["centroid"][2] == 1           # ties at -0.707: lowest valid index
    # the zero-norm centroid is not first: a zero-norm query still gets id 0 (nothing wins), not 1
    c2 = np.array([[1.0, 0.0], [0.0, 0.0], [0.0, 1.0]])
    out2 = oracle.route(np.array([[0.0, 0.0], [0.2, 1.0]]), c2)
    assert out2["centroid"][0] == 0 and np.isnan(out2["best"][0]) and out2["centroid"][1] == 2
    assert oracle.route(np.array([[1.0, 1.0]]), np.zeros((3, 2)))["centroid"][0] == 0   # all centroids zero
    one = oracle.route(np.array([[1.0, 2.0]]), np.array([[3.0, 1.0]]))
    assert one["centroid"][0] == 0 and np.isinf(one["margin"][0])


def test_planted_clusters_are_recovered():
    # Queries = cluster mean + 0.3 N(0, I), D = 768: the nearest centroid is the planted one.
    case = mi.planted_router(K=200, Q=256, D=768, seed=3)
    out = oracle.route(mi.bf16_bits(case.queries), mi.bf16_bits(case.centroids))
    assert np.array_equal(out["centroid"], case.labels.numpy())
    assert out["margin"].min() > 0.3
    # bf16 bit input == exactly widened double input
    out2 = oracle.route(mi.bf16_to_f64(case.queries), mi.bf16_to_f64(case.centroids))
    assert np.array_equal(out["centroid"], out2["centroid"])
    assert np.array_equal(out["best"], out2["best"])


def test_bucket_is_a_stable_grouping():
    rng = np.random.default_rng(6)
    slot = np.array([2, -1, 0, 1, -1, 3], np.int32)
    te = rng.integers(-1, 7, size=300).astype(np.int32)
    out = oracle.bucket(te, slot, 4)
    tok_slot = np.array([slot[e] if 0 <= e < 6 else -1 for e in te])
    key = np.where(tok_slot < 0, 1 << 20, tok_slot)
    assert np.array_equal(out["perm"], np.argsort(key, kind="stable"))   # library stable sort
    assert out["S"] == len(np.unique(tok_slot[tok_slot >= 0]))
    for s in range(out["S"]):
        seg = out["perm"][out["seg_start"][s]:out["seg_start"][s + 1]]
        assert np.all(tok_slot[seg] == out["seg_slot"][s]) and len(seg) > 0
    assert out["seg_start"][-1] == np.count_nonzero(tok_slot >= 0)
