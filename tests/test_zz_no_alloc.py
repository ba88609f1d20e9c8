"""moin_route_static: routing for callers that cannot allocate device memory (a worker whose memory
pool is frozen after start-up, a plug-in inside a foreign CUDA context).  Its scratch is a fixed array
inside the library, shared by all calls, so this file checks - through the C ABI - that it matches
moin_route on two calls in a row (the second call sees the first call's leftovers in the scratch),
that it agrees with the CPU oracle, that it really allocates nothing, and that it refuses batches beyond the
built-in limit.

Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest
import torch

import moin_inputs as mi
import oracle
import paper_2410_09687_b200 as moin

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(router, q):
    Q = q.shape[0]
    ref_e = torch.empty(Q, dtype=torch.int32, device=DEV)
    ref_c = torch.empty(Q, dtype=torch.int32, device=DEV)
    ref_b = torch.empty(Q, dtype=torch.float32, device=DEV)
    moin.route(router, q, out_expert=ref_e, out_centroid=ref_c, out_best_sim=ref_b)
    got_e, got_c, got_b = torch.empty_like(ref_e), torch.empty_like(ref_c), torch.empty_like(ref_b)
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    moin.route_static(router, q, got_e, got_c, got_b)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before       # no torch allocation on the way
    return (ref_e, ref_c, ref_b), (got_e, got_c, got_b)


def _assert_oracle(q, centroids, got_centroid, sample=None):
    """Ids against the fp64 oracle on the same bytes (all queries, or a seeded sample of them); queries whose two
    best cosines are closer than 1e-4 may legitimately differ."""
    rows = np.arange(q.shape[0]) if sample is None else np.sort(np.random.default_rng(5).choice(q.shape[0], sample, replace=False))
    ref = oracle.route(mi.bf16_bits(q[torch.as_tensor(rows, device=q.device)]), mi.bf16_bits(centroids))
    got = got_centroid.cpu().numpy()[rows]
    bad = (got != ref["centroid"]) & ~(ref["margin"] < 1e-4)
    assert not bad.any(), f"{int(bad.sum())} ids differ from the oracle outside near-ties"


def test_static_router_matches_workspace_router_twice_in_a_row():
    # first call: a large batch that fills most of the built-in scratch with winning keys
    big = mi.planted_router(K=1000, Q=40000, D=256, seed=11, device=DEV)
    cmap = torch.arange(1000, dtype=torch.int32, device=DEV).flip(0).contiguous()
    r_big = moin.Router(big.centroids, cmap)
    ref, got = _both(r_big, big.queries)
    assert torch.equal(ref[0], got[0]) and torch.equal(ref[1], got[1])     # ids: bit-exact
    assert torch.equal(got[1].cpu(), big.labels.cpu())
    np.testing.assert_allclose(got[2].cpu().numpy(), ref[2].cpu().numpy(), rtol=0, atol=0)
    _assert_oracle(big.queries, big.centroids, got[1], sample=2048)
    # second call right after, other table, fewer queries: stale keys of the first call must not leak
    small = mi.planted_router(K=300, Q=777, D=128, seed=12, device=DEV)
    r_small = moin.Router(small.centroids)
    ref2, got2 = _both(r_small, small.queries)
    assert torch.equal(ref2[0], got2[0]) and torch.equal(ref2[1], got2[1])
    assert torch.equal(got2[1].cpu(), small.labels.cpu())
    # both entry points pick the kernel by the same rule, so the cosines agree to the last bit as well
    np.testing.assert_allclose(got2[2].cpu().numpy(), ref2[2].cpu().numpy(), rtol=0, atol=0)
    _assert_oracle(small.queries, small.centroids, got2[1])
    assert moin.device_status()["timeout_flag"] == 0


def test_static_router_limits_and_small_dimension():
    case = mi.tiny_router(seed=0)                      # D = 64, 16 queries
    router = moin.Router(case.centroids.to(DEV))
    q = case.queries.to(DEV)
    out = torch.empty(16, dtype=torch.int32, device=DEV)
    moin.route_static(router, q, out)
    assert torch.equal(out, moin.route(router, q))
    too_many = torch.zeros(moin.ROUTE_STATIC_MAX_Q + 1, 64, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(moin.MoinError, match="WORKSPACE"):
        moin.route_static(router, too_many, torch.empty(too_many.shape[0], dtype=torch.int32, device=DEV))
    moin.route_static(router, q[:0], out[:0])          # empty batch: no-op
    # embedding dimension below the tensor-core kernel's minimum: the CUDA-core kernel, which needs no scratch
    low = mi.planted_router(K=40, Q=333, D=40, seed=13, device=DEV)
    r_low = moin.Router(low.centroids)
    ref, got = _both(r_low, low.queries)
    assert all(torch.equal(a, b) for a, b in zip(ref, got))
    _assert_oracle(low.queries, low.centroids, got[1])
    # forced tensor-core path on a decode-sized batch (the shape moin_route would give to the cluster kernel)
    moin.set_option(moin.OPT_GEMM_IMPL, 2)
    try:
        mid = mi.planted_router(K=500, Q=256, D=768, seed=14, device=DEV)
        r_mid = moin.Router(mid.centroids)
        ref, got = _both(r_mid, mid.queries)
        assert all(torch.equal(a, b) for a, b in zip(ref, got))
        _assert_oracle(mid.queries, mid.centroids, got[1])
    finally:
        moin.set_option(moin.OPT_GEMM_IMPL, 0)
