"""Router on the GPU against the oracle: ids bit-exact except near-ties (margin < 1e-4), which are counted."""
import numpy as np
import pytest
import torch

import moin_inputs as mi
import oracle
import paper_2410_09687_b200 as moin
from gpu_util import DEV, TIE_MARGIN, assert_router_matches

pytestmark = pytest.mark.gpu


def _route(case: mi.RouterCase, cmap=None, impl=0):
    moin.set_option(moin.OPT_GEMM_IMPL, impl)
    try:
        c, q = case.centroids.to(DEV), case.queries.to(DEV)
        m = None if cmap is None else torch.from_numpy(cmap).to(DEV)
        router = moin.Router(c, m)
        cid = torch.empty(case.Q, dtype=torch.int32, device=DEV)
        best = torch.empty(case.Q, dtype=torch.float32, device=DEV)
        eid = moin.route(router, q, out_centroid=cid, out_best_sim=best)
        torch.cuda.synchronize()
        return eid.cpu().numpy(), cid.cpu().numpy(), best.cpu().numpy()
    finally:
        moin.set_option(moin.OPT_GEMM_IMPL, 0)


def _oracle(case, cmap=None, rows=None):
    q = mi.bf16_bits(case.queries if rows is None else case.queries[torch.as_tensor(rows)])
    return oracle.route(q, mi.bf16_bits(case.centroids), cmap)


@pytest.mark.parametrize("impl", [0, 1])
def test_router_tiny(impl):
    case = mi.tiny_router(seed=0)
    eid, cid, best = _route(case, impl=impl)
    ref = _oracle(case)
    assert_router_matches(cid, ref)
    assert np.array_equal(eid, cid)
    np.testing.assert_allclose(best, ref["best"], atol=2e-3)


@pytest.mark.parametrize("impl", [0, 1, 2])   # 0: cluster kernel at this size, 1: CUDA cores, 2: tcgen05
def test_router_decode_shape_with_map(impl):
    case = mi.planted_router(K=500, Q=256, D=768, seed=1)
    cmap = np.arange(500, dtype=np.int32)[::-1].copy()
    cmap[::7] = -1
    eid, cid, best = _route(case, cmap, impl=impl)
    ref = _oracle(case, cmap)
    assert_router_matches(cid, ref)
    assert np.array_equal(eid, cmap[cid])
    assert np.array_equal(cid, case.labels.numpy())
    np.testing.assert_allclose(best, ref["best"], atol=2e-3)


def test_router_prefill_shape_5000_centroids():
    case = mi.planted_router(K=5000, Q=32, D=768, seed=2)
    _, cid, _ = _route(case)
    assert_router_matches(cid, _oracle(case))


def test_router_stress_full_size_sampled():
    # 65 536 x 5 000 x 768 on the GPU; the oracle checks a seeded sample of queries one by one.
    case = mi.planted_router(K=5000, Q=65536, D=768, seed=3, device=DEV)
    _, cid, _ = _route(case)
    assert np.array_equal(cid, case.labels.cpu().numpy())     # planted label (property at any size)
    rows = np.random.default_rng(0).choice(65536, size=1024, replace=False)
    host = mi.RouterCase(case.centroids.cpu(), case.queries.cpu(), None, case.K, case.D, case.Q)
    ref = _oracle(host, rows=rows)
    assert_router_matches(cid[rows], ref)


@pytest.mark.parametrize("Q,K,D", [(1, 1, 32), (33, 70, 64), (100, 17, 96), (257, 500, 768), (5, 5000, 768),
                                   (1024, 512, 256), (40, 1000, 1504)])
def test_router_small_batch_shapes(Q, K, D):
    # decode-sized batches (up to 1024 queries and 1024 centroids) take the single-launch cluster kernel:
    # ragged query groups, ragged centroid tiles, fewer tiles than warps in the cluster, two tiles per
    # warp; (5, 5000) is past the switch and takes the tensor-core GEMM
    case = mi.planted_router(K=K, Q=Q, D=D, seed=11 + Q)
    cmap = np.random.default_rng(Q).permutation(K).astype(np.int32)
    eid, cid, best = _route(case, cmap)
    ref = _oracle(case, cmap)
    assert_router_matches(cid, ref)
    assert np.array_equal(eid, cmap[cid])
    np.testing.assert_allclose(best, ref["best"], atol=2e-3)


def test_router_near_tie_stress():
    # noise added to the UNIT centroid: many small margins; mismatches only allowed below the margin.
    case = mi.planted_router(K=1000, Q=2048, D=768, seed=5, unit_centroid_noise=True)
    _, cid, _ = _route(case)
    ref = _oracle(case)
    n_near, n_diff = assert_router_matches(cid, ref)
    print(f"near-ties (<{TIE_MARGIN}): {n_near}, of which differ: {n_diff}")


@pytest.mark.parametrize("impl", [0, 1, 2])
def test_router_degenerate_inputs(impl):
    rng = np.random.default_rng(6)
    c = torch.from_numpy(rng.normal(size=(70, 64))).to(torch.bfloat16)
    c[3] = 0                       # zero-norm centroid: never chosen
    c[50] = c[10] * 4              # same direction as 10: exact tie in cosine up to rounding -> lowest index
    q = torch.from_numpy(rng.normal(size=(33, 64))).to(torch.bfloat16)
    q[0] = c[10]
    q[1] = c[3]                    # zero query
    case = mi.RouterCase(c, q, None, 70, 64, 33)
    _, cid, _ = _route(case, impl=impl)
    ref = _oracle(case)
    assert_router_matches(cid, ref)
    assert cid[0] in (10, 50) and cid[1] == 0 and 3 not in cid[2:]


def test_router_empty_batch():
    case = mi.tiny_router(seed=0)
    router = moin.Router(case.centroids.to(DEV))
    out = moin.route(router, torch.empty(0, 64, dtype=torch.bfloat16, device=DEV))
    assert out.numel() == 0


@pytest.mark.parametrize("impl", [1, 2])   # 1: CUDA cores, 2: tcgen05 with the two-slot key merge
@pytest.mark.parametrize("Q,K,D", [(300, 700, 768), (64, 1, 64), (1000, 5000, 128)])
def test_router_runner_up_and_margin(impl, Q, K, D):
    # best id as moin_route; the margin against the oracle's fp64 top-2 margin; the runner-up id is checked
    # through its cosine (cos(second) = cos(best) - margin), since equal runners-up are all correct
    case = mi.planted_router(K=K, Q=Q, D=D, seed=50 + K, unit_centroid_noise=True)
    moin.set_option(moin.OPT_GEMM_IMPL, impl)
    try:
        router = moin.Router(case.centroids.to(DEV))
        out = {k: v.cpu().numpy() for k, v in moin.route_top2(router, case.queries.to(DEV)).items()}
    finally:
        moin.set_option(moin.OPT_GEMM_IMPL, 0)
    ref = _oracle(case)
    assert_router_matches(out["centroid"], ref)
    assert np.array_equal(out["expert"], out["centroid"])
    np.testing.assert_allclose(out["best"], ref["best"], atol=2e-3)
    if K == 1:
        assert (out["second"] == -1).all() and np.isinf(out["margin"]).all()
        return
    tol = 2e-5 + 2e-3 * np.abs(ref["margin"])
    assert (np.abs(out["margin"] - ref["margin"]) <= tol).all(), np.abs(out["margin"] - ref["margin"]).max()
    c = mi.bf16_to_f64(case.centroids)
    q = mi.bf16_to_f64(case.queries)
    cos2 = (q * c[out["second"]]).sum(1) / (np.linalg.norm(q, axis=1) * np.linalg.norm(c[out["second"]], axis=1))
    assert (np.abs(cos2 - (ref["best"] - ref["margin"])) <= tol).all()
    assert (out["second"] != out["centroid"]).all()
    assert moin.device_status()["timeout_flag"] == 0
