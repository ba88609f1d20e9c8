"""K-means iteration on the GPU (route -> plan -> moin_kmeans_update) against the oracle.

The update adds bf16 inputs in fp32, in member order, and rounds the mean once to bf16: against the fp64 mean
that is half a bf16 ulp (8 significand bits: at most 2^-8 = 3.906e-3 relative) plus the fp32 accumulation error
(~1e-7 per addend), so |delta| <= 3.95e-3 |ref| + 1e-6 max|ref| is the bound used here.  Assignments are integer work: bit-exact except near-ties of the router (< 1e-4)."""
import numpy as np
import pytest
import torch

import moin_inputs as mi
import oracle
import paper_2410_09687_b200 as moin
from gpu_util import DEV, assert_router_matches

pytestmark = pytest.mark.gpu


def _assert_centroids_close(got_bf16: torch.Tensor, want: np.ndarray, what: str):
    got = mi.bf16_to_f64(got_bf16)
    tol = 3.95e-3 * np.abs(want) + 1e-6 * np.abs(want).max()
    bad = np.abs(got - want) > tol
    assert not bad.any(), f"{what}: {int(bad.sum())} elements off, worst {np.abs(got - want).max():.3e}"


def _gpu_update(x, c_old, assign_np, K):
    plan = moin.plan_build(torch.from_numpy(assign_np.astype(np.int32)).to(DEV), K, moin.PLAN_SEGMENTS)
    inv = torch.empty(K, dtype=torch.float32, device=DEV)
    c_new = moin.kmeans_update(plan, x.to(DEV), c_old.to(DEV), inv_norm_new=inv)
    torch.cuda.synchronize()
    return c_new, inv


@pytest.mark.parametrize("N,K,D", [(5000, 300, 768), (777, 40, 64), (1000, 1000, 136), (4096, 3, 2048), (9, 16, 8)])
def test_update_matches_the_oracle(N, K, D):
    rng = mi.np_rng(31, N)
    x = mi.normal_bf16((N, D), 1.0, 31, N, 1)
    c_old = mi.normal_bf16((K, D), 1.0, 31, N, 2)
    assign = rng.integers(-1, K, size=N)          # -1: point without a cluster
    if K > 8:
        assign[assign == 5] = 6                   # cluster 5 stays empty
    c_new, inv = _gpu_update(x, c_old, assign, K)
    ref = oracle.kmeans_update(mi.bf16_bits(x), mi.bf16_bits(c_old), assign)
    _assert_centroids_close(c_new, ref["centroids"], f"update {N}x{K}x{D}")
    empty = ref["counts"] == 0
    assert torch.equal(c_new[torch.from_numpy(empty).to(DEV)], c_old.to(DEV)[torch.from_numpy(empty).to(DEV)])
    # the inverse norms are those of the stored (bf16) new centroids
    norms = np.linalg.norm(mi.bf16_to_f64(c_new), axis=1)
    np.testing.assert_allclose(inv.cpu().numpy(), 1.0 / norms, rtol=2e-6)


def test_in_place_update_and_empty_batch():
    x = mi.normal_bf16((600, 64), 1.0, 32, 1)
    c = mi.normal_bf16((10, 64), 1.0, 32, 2).to(DEV)
    assign = mi.np_rng(32, 3).integers(0, 7, size=600)          # clusters 7..9 empty
    ref = oracle.kmeans_update(mi.bf16_bits(x), mi.bf16_bits(c), assign)
    plan = moin.plan_build(torch.from_numpy(assign.astype(np.int32)).to(DEV), 10, moin.PLAN_SEGMENTS)
    out = moin.kmeans_update(plan, x.to(DEV), c, centroids_new=c)
    torch.cuda.synchronize()
    assert out.data_ptr() == c.data_ptr()
    _assert_centroids_close(c, ref["centroids"], "in place")
    plan0 = moin.Plan(0, 10, DEV, moin.PLAN_SEGMENTS)
    kept = moin.kmeans_update(plan0, torch.empty(0, 64, dtype=torch.bfloat16, device=DEV), c)
    torch.cuda.synchronize()
    assert torch.equal(kept, c)
    with pytest.raises(moin.MoinError, match="BAD_SHAPE"):
        moin.kmeans_update(moin.Plan(4, 10, DEV), torch.zeros(4, 12, dtype=torch.bfloat16, device=DEV),
                           torch.zeros(10, 12, dtype=torch.bfloat16, device=DEV))


def test_lloyd_iterations_on_planted_clusters():
    # every iteration is checked teacher-forced: the oracle is fed the GPU's own centroids of the step before
    K, N, D = 200, 20000, 768
    rc = mi.planted_router(K=K, Q=N, D=D, seed=33, noise=0.3)
    x = rc.queries.to(DEV)
    xb = mi.bf16_bits(rc.queries)
    g = torch.Generator().manual_seed(5)
    c = (rc.centroids.float() + 0.4 * torch.randn(K, D, generator=g) / D ** 0.5).to(torch.bfloat16).to(DEV)
    assign = torch.empty(N, dtype=torch.int32, device=DEV)
    plan = moin.Plan(N, K, DEV, moin.PLAN_SEGMENTS)
    last = -np.inf
    for it in range(4):
        router = moin.Router(c)
        moin.route(router, x, out_expert=assign)
        moin.plan_build(assign, K, moin.PLAN_SEGMENTS, plan=plan)
        c_new = moin.kmeans_update(plan, x, c)
        torch.cuda.synchronize()
        ref_assign = oracle.route(xb, mi.bf16_bits(c))
        a = assign.cpu().numpy()
        assert_router_matches(a, ref_assign)
        ref = oracle.kmeans_update(xb, mi.bf16_bits(c), a)       # same assignment, same old centroids
        _assert_centroids_close(c_new, ref["centroids"], f"iteration {it}")
        obj = float(ref_assign["best"].sum())                    # summed cosine to the assigned centroid
        assert obj >= last - 1e-6 * N
        last = obj
        c = c_new
    planted = mi.bf16_to_f64(rc.centroids)
    got = mi.bf16_to_f64(c)
    cos = (got * planted).sum(1) / (np.linalg.norm(got, axis=1) * np.linalg.norm(planted, axis=1))
    assert cos.min() > 0.99
    assert moin.device_status()["timeout_flag"] == 0
