"""Support features around the hot path: replacing one expert's adapter in a resident pool, guard rows around every
output (nothing is written outside the rows a call owns), and the NVTX option."""
import numpy as np
import pytest
import torch

import moin_inputs as mi
import oracle
import paper_2410_09687_b200 as moin
from gpu_util import DEV, assert_layer_close, gpu_pool

pytestmark = pytest.mark.gpu
MODES = [moin.PLAN_SEGMENTS, moin.PLAN_TILES]


@pytest.mark.parametrize("mode", MODES)
def test_pool_set_adapter_replaces_one_expert(mode):
    """A retrained expert is written into its slot and an adapter-less expert gets one (Sec. 1 / Sec. 5: experts are
    added or replaced independently); calls issued afterwards on the stream use the new adapters."""
    rng = mi.np_rng(51, 1)
    E, r, d_in, d_out, T = 8, 16, 256, 200, 300
    pool = mi.make_pool(E, r, d_in, d_out, 51, 2, missing=(3,))
    lens = rng.multinomial(T - 6, [1 / 6] * 6) + 1
    te = np.repeat(np.array([0, 3, 5, 3, 7, 0]), lens).astype(np.int32) if mode == moin.PLAN_TILES else \
        rng.integers(-1, E, size=T).astype(np.int32)
    case = mi.layer_case("upd", len(te), d_in, d_out, pool, te, 2.0, 51, 3)
    gp = gpu_pool(pool)
    x, W = case.x.to(DEV), case.W.to(DEV)
    plan = moin.plan_build(torch.from_numpy(te).to(DEV), E, mode)
    A, B, so = pool.A.clone(), pool.B.clone(), pool.slot_of_expert.clone()

    def ref():
        return oracle.lora_linear(mi.bf16_bits(case.x), mi.bf16_bits(case.W), mi.bf16_bits(A), mi.bf16_bits(B), te, so.numpy(), 2.0)

    assert_layer_close(moin.lora_linear(plan, x, W, gp, 2.0), ref(), "before")
    # expert 5 retrained (from device memory), expert 3 gets the free slot... there is none: it takes over expert 7's
    newA = mi.normal_bf16((r, d_in), 0.02, 51, 9)
    newB = mi.normal_bf16((d_out, r), 0.02, 51, 10)
    s5, s7 = int(so[5]), int(so[7])
    moin.pool_set_adapter(gp, 5, s5, newA.to(DEV), newB.to(DEV))
    A[s5], B[s5] = newA, newB
    hA, hB = mi.normal_bf16((r, d_in), 0.02, 51, 11).pin_memory(), mi.normal_bf16((d_out, r), 0.02, 51, 12).pin_memory()
    moin.pool_set_adapter(gp, 7, -1)                       # unmap 7 ...
    moin.pool_set_adapter(gp, 3, s7, hA, hB)               # ... and give its slot to 3, from pinned host memory
    so[7], so[3] = -1, s7
    A[s7], B[s7] = hA, hB
    y = moin.lora_linear(plan, x, W, gp, 2.0)
    torch.cuda.synchronize()
    assert torch.equal(gp.slot_of_expert.cpu(), so)
    assert_layer_close(y, ref(), "after")
    with pytest.raises(moin.MoinError, match="INVALID_ARG"):
        moin.pool_set_adapter(gp, E, 0, newA.to(DEV), newB.to(DEV))
    with pytest.raises(moin.MoinError, match="INVALID_ARG"):
        moin.pool_set_adapter(gp, 0, gp.n_slots, newA.to(DEV), newB.to(DEV))


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("shape", [(333, 192, 328, 24), (256, 2048, 256, 64), (130, 512, 72, 128)])
def test_guard_rows_around_outputs_stay_untouched(mode, shape):
    """y lives inside a larger buffer filled with a marker: the rows before and after it (and the workspace's tail)
    must come back unchanged - no kernel writes outside [T, d_out]."""
    T, d_in, d_out, r = shape
    rng = mi.np_rng(53, T)
    E = 7
    pool = mi.make_pool(E, r, d_in, d_out, 53, T, missing=(2,))
    te = rng.integers(-1, E, size=T).astype(np.int32) if mode == moin.PLAN_SEGMENTS else \
        np.repeat(rng.integers(0, E, size=3), [T - 2 * (T // 3), T // 3, T // 3]).astype(np.int32)
    case = mi.layer_case("guard", T, d_in, d_out, pool, te, 2.0, 53, 3)
    G = 4
    marker = torch.tensor(-12345.0, dtype=torch.bfloat16)
    big = torch.full((T + 2 * G, d_out), float(marker), dtype=torch.bfloat16, device=DEV)
    y = big[G:G + T]
    n = moin.lib().moin_lora_linear_workspace_bytes(T, d_in, d_out, r)
    ws = torch.full((n + 4096,), 0x5A, dtype=torch.uint8, device=DEV)
    plan = moin.plan_build(torch.from_numpy(te).to(DEV), E, mode)
    moin.lora_linear(plan, case.x.to(DEV), case.W.to(DEV), gpu_pool(pool), 2.0, y=y, workspace=ws[:n])
    torch.cuda.synchronize()
    assert (big[:G] == marker).all() and (big[G + T:] == marker).all()
    assert (ws[n:] == 0x5A).all()
    ref = oracle.lora_linear(mi.bf16_bits(case.x), mi.bf16_bits(case.W), mi.bf16_bits(pool.A), mi.bf16_bits(pool.B), te,
                             pool.slot_of_expert.numpy(), 2.0)
    assert_layer_close(y, ref, "guarded")


def test_nvtx_option_leaves_results_unchanged():
    case = mi.tiny_layer(seed=0)
    gp = gpu_pool(case.pool)
    plan = moin.plan_build(case.token_expert.to(DEV), case.pool.E, moin.PLAN_SEGMENTS)
    y0 = moin.lora_linear(plan, case.x.to(DEV), case.W.to(DEV), gp, case.scale).clone()
    moin.set_option(moin.OPT_NVTX, 1)
    try:
        y1 = moin.lora_linear(plan, case.x.to(DEV), case.W.to(DEV), gp, case.scale)
        torch.cuda.synchronize()
    finally:
        moin.set_option(moin.OPT_NVTX, 0)
    assert torch.equal(y0, y1)
    with pytest.raises(moin.MoinError, match="INVALID_ARG"):
        moin.set_option(moin.OPT_NVTX, 7)
