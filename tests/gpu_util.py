"""Helpers shared by the GPU parity tests: move seeded cases to the device, call the C-ABI
binding, run the oracle on the same bytes, and apply the stated tolerances."""
import numpy as np
import torch

import moin_inputs as mi
import oracle
import paper_2410_09687_b200 as moin

DEV = "cuda:0"
# Tolerances of the routed layer (bf16 inputs, fp32 accumulate, one bf16 rounding at the output):
REL_FRO = 5e-3        # relative Frobenius error
ELEM_TOL = 2e-2       # |d| <= ELEM_TOL * (1 + |ref|)
TIE_MARGIN = 1e-4     # router: queries whose top-2 cosine margin is below this may differ


def gpu_pool(pool: mi.AdapterPool) -> moin.Pool:
    return moin.Pool(pool.A.to(DEV), pool.B.to(DEV), pool.slot_of_expert.to(DEV))


def compact_pool_for(pool: mi.AdapterPool, token_expert: np.ndarray):
    """Host copies of only the adapters the given tokens use, with a remapped slot table."""
    so = pool.slot_of_expert.cpu().numpy()
    used = sorted({int(so[e]) for e in token_expert if 0 <= e < pool.E and so[e] >= 0})
    remap = {s: i for i, s in enumerate(used)}
    so2 = np.array([remap.get(int(s), -1) if s >= 0 else -1 for s in so], np.int32)
    idx = torch.tensor(used if used else [0], dtype=torch.long, device=pool.A.device)
    return mi.bf16_bits(pool.A[idx]), mi.bf16_bits(pool.B[idx]), so2


def oracle_layer(case: mi.LayerCase, rows=None) -> np.ndarray:
    te = case.token_expert.cpu().numpy()
    rows = np.arange(case.T) if rows is None else np.asarray(rows)
    A, B, so = compact_pool_for(case.pool, te[rows])
    x = mi.bf16_bits(case.x[torch.as_tensor(rows, device=case.x.device)])
    return oracle.lora_linear(x, mi.bf16_bits(case.W), A, B, te[rows], so, case.scale)


def assert_layer_close(y_gpu: torch.Tensor, ref: np.ndarray, what=""):
    got = y_gpu.detach().to(torch.float64).cpu().numpy()
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    viol = np.abs(got - ref) > ELEM_TOL * (1.0 + np.abs(ref))
    assert rel <= REL_FRO, f"{what}: relative Frobenius error {rel:.3e} > {REL_FRO}"
    assert not viol.any(), f"{what}: {int(viol.sum())} elements beyond |d| <= {ELEM_TOL}(1+|ref|)"
    return rel


def run_layer(case: mi.LayerCase, mode=moin.PLAN_AUTO, pool=None, plan=None):
    x, W, te = case.x.to(DEV), case.W.to(DEV), case.token_expert.to(DEV)
    pool = gpu_pool(case.pool) if pool is None else pool
    plan = moin.plan_build(te, case.pool.E, mode) if plan is None else plan
    y = moin.lora_linear(plan, x, W, pool, case.scale)
    torch.cuda.synchronize()
    return y, plan


def assert_router_matches(ids_gpu: np.ndarray, ref: dict, key="centroid"):
    """Bit-exact ids except near-ties (top-2 margin < TIE_MARGIN), which are counted and returned."""
    diff = ids_gpu != ref[key]
    near = ref["margin"] < TIE_MARGIN
    bad = diff & ~near
    assert not bad.any(), f"{int(bad.sum())} router mismatches outside near-ties, e.g. query {np.nonzero(bad)[0][:5]}"
    return int(near.sum()), int((diff & near).sum())
