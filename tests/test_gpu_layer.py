"""Routed LoRA linear layer on the GPU against the fp64 oracle (Sec. 3.2 formula, expert per token)."""
import numpy as np
import pytest
import torch

import moin_inputs as mi
import oracle
import paper_2410_09687_b200 as moin
from gpu_util import compact_pool_for, DEV, assert_layer_close, gpu_pool, oracle_layer, run_layer

pytestmark = pytest.mark.gpu
MODES = [moin.PLAN_SEGMENTS, moin.PLAN_TILES]


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("impl", [0, 1])
def test_tiny_config(mode, impl):
    moin.set_option(moin.OPT_GEMM_IMPL, impl)
    try:
        case = mi.tiny_layer(seed=0)
        y, _ = run_layer(case, mode)
        assert_layer_close(y, oracle_layer(case), "tiny")
    finally:
        moin.set_option(moin.OPT_GEMM_IMPL, 0)


def test_tiny_config_routed_by_the_router():
    # the router's ids feed the layer: 16 requests, each routed to one of 8 experts
    rc = mi.tiny_router(seed=0)
    case = mi.tiny_layer(seed=0)
    router = moin.Router(rc.centroids.to(DEV))
    req_expert = moin.route(router, rc.queries.to(DEV)).cpu().numpy()
    ref_ids = oracle.route(mi.bf16_bits(rc.queries), mi.bf16_bits(rc.centroids))["expert"]
    assert np.array_equal(req_expert, ref_ids)
    case.token_expert = torch.from_numpy(mi.expand_request_experts(req_expert, case.lengths))
    y, _ = run_layer(case)
    assert_layer_close(y, oracle_layer(case), "tiny routed")


@pytest.mark.parametrize("r", [8, 16, 24, 32, 40, 48, 56, 64, 72, 96, 120, 128])
@pytest.mark.parametrize("mode", MODES)
def test_every_supported_rank(r, mode):
    rng = mi.np_rng(7, r)
    # ragged T, d_out not a multiple of 16 or 64; d_in alternates between a multiple of 256 and not
    E, T, d_in, d_out = 6, 333, (192 if r % 16 else 512), 328
    pool = mi.make_pool(E, r, d_in, d_out, 7, r, missing=(4,))
    lens = rng.multinomial(T - 8, [1 / 8] * 8) + 1
    te = np.repeat(rng.integers(-1, E, size=8), lens).astype(np.int32)
    case = mi.layer_case("ranks", T, d_in, d_out, pool, te, 2.0, 7, r)
    y, _ = run_layer(case, mode)
    assert_layer_close(y, oracle_layer(case), f"rank {r}")


@pytest.mark.parametrize("mode", MODES)
def test_base_only_and_missing_adapters(mode):
    pool = mi.make_pool(5, 16, 256, 128, 8, 1, missing=(1, 3))
    te = np.array([-1, 1, 3, 0, 2, 4, 99, -5] * 20, np.int32)
    case = mi.layer_case("fallback", len(te), 256, 128, pool, te, 2.0, 8, 2)
    y, _ = run_layer(case, mode)
    ref = oracle_layer(case)
    assert_layer_close(y, ref, "fallback")
    # tokens without an adapter equal the base layer computed by the same library
    y_base = moin.lora_linear(None, case.x.to(DEV), case.W.to(DEV), None, 0.0)
    so = pool.slot_of_expert.numpy()
    base_rows = np.array([not (0 <= e < 5 and so[e] >= 0) for e in te])
    assert torch.equal(y[torch.from_numpy(base_rows).to(DEV)], y_base[torch.from_numpy(base_rows).to(DEV)])
    assert_layer_close(y_base, oracle.lora_linear(mi.bf16_bits(case.x), mi.bf16_bits(case.W), None, None, None,
                                                  None, 0.0), "base")


def test_decode_shape_at_the_papers_rank_128():
    # Sec. 4 trains every expert at rank 128: 256 single-token requests over 120 such experts, a wide projection
    E, r, T, d_in, d_out = 120, 128, 256, 2048, 2048
    pool = mi.make_pool(E, r, d_in, d_out, 21, 1)
    te = mi.np_rng(21, 2).integers(0, E, size=T).astype(np.int32)
    case = mi.layer_case("rank128", T, d_in, d_out, pool, te, 2.0, 21, 3)
    y, _ = run_layer(case, moin.PLAN_SEGMENTS)
    assert_layer_close(y, oracle_layer(case), "rank 128 decode")


def test_long_runs_at_rank_128_through_the_fused_gemm():
    # 8 requests x 256 tokens, full-width projection: the rank spans two 64-wide blocks of the appended K range
    E, r, d_in, d_out = 16, 128, 2048, 2048
    pool = mi.make_pool(E, r, d_in, d_out, 22, 1, missing=(5,))
    req = np.array([3, 7, 5, 0, -1, 15, 7, 2], np.int32)
    te = np.repeat(req, 256).astype(np.int32)
    case = mi.layer_case("rank128 runs", len(te), d_in, d_out, pool, te, 2.0, 22, 3)
    y, _ = run_layer(case, moin.PLAN_TILES)
    assert_layer_close(y, oracle_layer(case), "rank 128 long runs")


def test_decode_config_all_projections():
    # 256 single-token requests, 500 rank-64 experts: every token checked against the oracle.
    cases = mi.decode_batch(seed=1, device=DEV)
    te = cases[0].token_expert
    plan = moin.plan_build(te.to(DEV), 500, moin.PLAN_SEGMENTS)
    for case in cases:
        y, _ = run_layer(case, plan=plan)
        rel = assert_layer_close(y, oracle_layer(case), f"decode {case.name}")
        print(f"decode {case.name}: rel Frobenius {rel:.2e}")
    del cases
    torch.cuda.empty_cache()


def test_prefill_config_sampled_rows():
    # 32 x 512 tokens, 5 000 rank-16 experts, Zipf-skewed: 64 seeded rows per projection against the oracle.
    cases = mi.prefill_batch(seed=2, device=DEV)
    plan = moin.plan_build(cases[0].token_expert.to(DEV), 5000, moin.PLAN_AUTO)
    rows = np.sort(np.random.default_rng(0).choice(cases[0].T, size=64, replace=False))
    for case in cases:
        y, _ = run_layer(case, plan=plan)
        ref = oracle_layer(case, rows)
        assert_layer_close(y[torch.from_numpy(rows).to(DEV)], ref, f"prefill {case.name}")
    del cases
    torch.cuda.empty_cache()


@pytest.mark.parametrize("mode", MODES)
def test_request_permutation_and_determinism(mode):
    # experts do not interact: permuting requests permutes output rows (bitwise), and reruns are bitwise equal
    pool = mi.make_pool(12, 32, 256, 256, 9, 1)
    rng = mi.np_rng(9, 2)
    req = rng.integers(0, 12, size=10)
    L = 160
    te = np.repeat(req, L).astype(np.int32)
    case = mi.layer_case("perm", len(te), 256, 256, pool, te, 2.0, 9, 3)
    gp = gpu_pool(pool)
    y1, _ = run_layer(case, mode, pool=gp)
    y2, _ = run_layer(case, mode, pool=gp)
    assert torch.equal(y1, y2)
    p = rng.permutation(10)
    rows = np.concatenate([np.arange(i * L, (i + 1) * L) for i in p])
    case_p = mi.LayerCase("perm2", case.x[torch.from_numpy(rows)], case.W, pool, torch.from_numpy(te[rows]), 2.0,
                          len(te))
    y3, _ = run_layer(case_p, mode, pool=gp)
    assert torch.equal(y3, y1[torch.from_numpy(rows).to(DEV)])


@pytest.mark.parametrize("mode", MODES)
def test_grouped_projections_equal_single_calls(mode):
    # {q,k,v}-like group: shared plan, different shapes; the group's outputs are bit-identical to one call per
    # projection, and match the oracle.
    rng = mi.np_rng(13, 1)
    E, T = 40, 200
    te = rng.integers(-1, E, size=T).astype(np.int32) if mode == moin.PLAN_SEGMENTS else \
        np.repeat(rng.integers(0, E, size=2), [130, 70]).astype(np.int32)
    shapes = [(512, 512, 32), (512, 64, 32), (512, 72, 16), (256, 1024, 64)]
    plan = moin.plan_build(torch.from_numpy(te).to(DEV), E, mode)
    cases, jobs, singles = [], [], []
    for i, (d_in, d_out, r) in enumerate(shapes):
        pool = mi.make_pool(E, r, d_in, d_out, 13, 10 + i, missing=(3,))
        case = mi.layer_case(f"g{i}", T, d_in, d_out, pool, te, 2.0, 13, 20 + i)
        gp = gpu_pool(pool)
        x, W = case.x.to(DEV), case.W.to(DEV)
        y = torch.empty(T, d_out, dtype=torch.bfloat16, device=DEV)
        cases.append(case)
        jobs.append((x, W, gp, y))
        singles.append(moin.lora_linear(plan, x, W, gp, 2.0).clone())
    moin.lora_linear_group(plan, moin.JobGroup(jobs), 2.0)
    torch.cuda.synchronize()
    for case, (x, W, gp, y), y1 in zip(cases, jobs, singles):
        assert torch.equal(y, y1), case.name
        assert_layer_close(y, oracle_layer(case), case.name)


@pytest.mark.parametrize("r,n_proj", [(16, 3), (32, 3), (64, 2), (64, 3), (128, 2)])
def test_grouped_projections_that_share_their_input(r, n_proj):
    """{q, k, v} / {gate, up}-like groups over long runs: the projections read the SAME x, so their shrinks are one
    pass over it with the adapters' rows side by side in one tile (where n_proj * r fits: up to 256).  Every pool
    misses a different expert and gives its slots different ranks; each output must be bit-identical to the
    single call and match the oracle."""
    rng = mi.np_rng(29, r)
    E, T, d_in = 12, 300, 256
    te = np.repeat(rng.integers(0, E, size=4), [130, 70, 37, 63]).astype(np.int32)
    te[5:9] = -1
    plan = moin.plan_build(torch.from_numpy(te).to(DEV), E, moin.PLAN_TILES)
    x = mi.normal_bf16((T, d_in), 1.0, 29, r, 1).to(DEV)
    jobs, refs, singles = [], [], []
    for i in range(n_proj):
        d_out = [256, 64, 136][i]
        pool = mi.make_pool(E, r, d_in, d_out, 29, 10 + i, missing=(int(te[0]) if i == 1 else (i + 2) % E,))
        n_slots = pool.A.shape[0]
        ranks = np.array([[r, 8, r // 2, 0][(s_ + i) % 4] for s_ in range(n_slots)], np.int32)
        W = mi.normal_bf16((d_out, d_in), 0.05, 29, r, 20 + i)
        gp = moin.Pool(pool.A.to(DEV), pool.B.to(DEV), pool.slot_of_expert.to(DEV), slot_rank=torch.from_numpy(ranks).to(DEV))
        y = torch.empty(T, d_out, dtype=torch.bfloat16, device=DEV)
        jobs.append((x, W.to(DEV), gp, y))
        singles.append(moin.lora_linear(plan, x, W.to(DEV), gp, 2.0).clone())
        refs.append(oracle.lora_linear(mi.bf16_bits(x.cpu()), mi.bf16_bits(W), mi.bf16_bits(pool.A), mi.bf16_bits(pool.B), te,
                                       pool.slot_of_expert.numpy(), 2.0, slot_rank=ranks))
    moin.lora_linear_group(plan, moin.JobGroup(jobs), 2.0)
    torch.cuda.synchronize()
    assert moin.device_status()["timeout_flag"] == 0
    for i, ((_, _, _, y), y1, ref) in enumerate(zip(jobs, singles, refs)):
        assert torch.equal(y, y1), i
        assert_layer_close(y, ref, f"shared input, projection {i}")


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_seeded_random_shapes_in_every_plan_mode(seed):
    # ranks, widths (also not multiples of 16 / 64), segment structures (runs, interleaved tokens, base-only
    # tokens, out-of-range ids, experts without adapters) drawn at random; every mode against the oracle
    rng = np.random.default_rng(seed)
    for it in range(10):
        r = int(rng.choice([8, 16, 24, 40, 64, 72, 128]))
        d_in = int(rng.choice([64, 128, 192, 256, 320, 512, 1024, 2048]))
        d_out = int(rng.choice([8, 24, 64, 72, 136, 256, 328, 512, 1000, 2048]))
        E = int(rng.integers(1, 40))
        n_req = int(rng.integers(1, 24))
        lens = rng.integers(1, int(rng.choice([1, 3, 9, 40, 200])) + 1, size=n_req)
        te = np.repeat(rng.integers(-1, E, size=n_req), lens).astype(np.int32)
        if rng.random() < 0.3:
            te = rng.permutation(te)
        if rng.random() < 0.2:
            te[rng.integers(0, len(te))] = E + 5
        missing = tuple(int(m) for m in rng.choice(E, size=min(E - 1, int(rng.integers(0, 3))), replace=False)) if E > 1 else ()
        pool = mi.make_pool(E, r, d_in, d_out, 100 * seed + it, 1, missing=missing)
        case = mi.layer_case("random", len(te), d_in, d_out, pool, te, float(rng.choice([1.0, 2.0, 0.5])), 100 * seed + it, 2)
        ref = oracle_layer(case)
        for mode in (moin.PLAN_SEGMENTS, moin.PLAN_TILES, moin.PLAN_AUTO):
            y, _ = run_layer(case, mode)
            assert_layer_close(y, ref, f"seed {seed} case {it} mode {mode}: r {r}, {d_in}->{d_out}, E {E}, T {len(te)}")


def _variant_case(seed, mode, r, T=300, E=12, d_in=512, d_out=328):
    rng = mi.np_rng(seed, 1)
    pool = mi.make_pool(E, r, d_in, d_out, seed, 2, missing=(5,))
    if mode == moin.PLAN_SEGMENTS:
        te = rng.integers(-1, E, size=T).astype(np.int32)
    else:
        lens = rng.multinomial(T - 6, [1 / 6] * 6) + 1
        te = np.repeat(rng.integers(0, E, size=6), lens).astype(np.int32)
    return pool, mi.layer_case("variant", len(te), d_in, d_out, pool, te, 2.0, seed, 3), te


@pytest.mark.parametrize("act", [moin.ACT_RELU, moin.ACT_SILU, moin.ACT_GELU])
@pytest.mark.parametrize("mode", MODES)
def test_activation_between_the_low_rank_matrices(act, mode):
    """y = W x + s W_b act(W_a x) (the paper's future-work variant, Sec. 5) against the oracle, both plan modes."""
    pool, case, te = _variant_case(31, mode, 40)
    gp = moin.Pool(pool.A.to(DEV), pool.B.to(DEV), pool.slot_of_expert.to(DEV), activation=act)
    y, _ = run_layer(case, mode, pool=gp)
    A, B, so = compact_pool_for(pool, te)
    ref = oracle.lora_linear(mi.bf16_bits(case.x), mi.bf16_bits(case.W), A, B, te, so, case.scale, act=act)
    assert_layer_close(y, ref, f"activation {act}")
    plain = oracle.lora_linear(mi.bf16_bits(case.x), mi.bf16_bits(case.W), A, B, te, so, case.scale)
    assert np.linalg.norm(ref - plain) / np.linalg.norm(plain) > 0.02    # the activation is not a no-op here


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("r", [64, 128])
def test_mixed_rank_pool(mode, r):
    """A rank per slot (the paper's future-work "adaptive rank", Sec. 5): pools storing rank r whose slots use
    8 ... r of it.  What is stored beyond a slot's rank is large finite garbage: it must not reach the result."""
    pool, case, te = _variant_case(37, mode, r)
    n_slots = pool.A.shape[0]
    ranks = np.array([[8, 16, r, 24, r // 2, 0][i % 6] for i in range(n_slots)], np.int32)
    A, B = pool.A.clone(), pool.B.clone()
    for s_, k in enumerate(ranks):
        A[s_, k:, :] = 3.0e38
        B[s_, :, k:] = -3.0e38
    gp = moin.Pool(A.to(DEV), B.to(DEV), pool.slot_of_expert.to(DEV), slot_rank=torch.from_numpy(ranks).to(DEV))
    y, _ = run_layer(case, mode, pool=gp)
    ref = oracle.lora_linear(mi.bf16_bits(case.x), mi.bf16_bits(case.W), mi.bf16_bits(A), mi.bf16_bits(B), te,
                             pool.slot_of_expert.numpy(), case.scale, slot_rank=ranks)
    assert_layer_close(y, ref, f"mixed ranks, stored {r}")
    # with activation on top, and against the uniform-rank result to see that the ranks matter
    gp2 = moin.Pool(A.to(DEV), B.to(DEV), pool.slot_of_expert.to(DEV), slot_rank=torch.from_numpy(ranks).to(DEV),
                    activation=moin.ACT_SILU)
    y2, _ = run_layer(case, mode, pool=gp2)
    ref2 = oracle.lora_linear(mi.bf16_bits(case.x), mi.bf16_bits(case.W), mi.bf16_bits(A), mi.bf16_bits(B), te,
                              pool.slot_of_expert.numpy(), case.scale, slot_rank=ranks, act=oracle.ACT_SILU)
    assert_layer_close(y2, ref2, f"mixed ranks + SiLU, stored {r}")
    full = oracle.lora_linear(mi.bf16_bits(case.x), mi.bf16_bits(case.W), mi.bf16_bits(pool.A), mi.bf16_bits(pool.B), te,
                              pool.slot_of_expert.numpy(), case.scale)
    assert np.linalg.norm(ref - full) / np.linalg.norm(full) > 0.02


def test_empty_batch_and_argument_errors():
    pool = gpu_pool(mi.make_pool(4, 8, 64, 64, 10, 1))
    x = torch.zeros(0, 64, dtype=torch.bfloat16, device=DEV)
    W = torch.zeros(64, 64, dtype=torch.bfloat16, device=DEV)
    plan = moin.plan_build(torch.zeros(0, dtype=torch.int32, device=DEV), 4, moin.PLAN_SEGMENTS)
    assert moin.lora_linear(plan, x, W, pool, 1.0).shape == (0, 64)
    bad = moin.Pool(torch.zeros(4, 12, 64, dtype=torch.bfloat16, device=DEV),
                    torch.zeros(4, 64, 12, dtype=torch.bfloat16, device=DEV), pool.slot_of_expert)
    x1 = torch.zeros(8, 64, dtype=torch.bfloat16, device=DEV)
    plan1 = moin.plan_build(torch.zeros(8, dtype=torch.int32, device=DEV), 4, moin.PLAN_SEGMENTS)
    with pytest.raises(moin.MoinError, match="UNSUPPORTED_RANK"):
        moin.lora_linear(plan1, x1, W, bad, 1.0)
    with pytest.raises(moin.MoinError, match="BAD_SHAPE"):
        moin.lora_linear(None, torch.zeros(8, 40, dtype=torch.bfloat16, device=DEV),
                         torch.zeros(64, 40, dtype=torch.bfloat16, device=DEV), None, 1.0)
    with pytest.raises(moin.MoinError, match="MISALIGNED"):
        buf = torch.zeros(8 * 64 + 8, dtype=torch.bfloat16, device=DEV)
        moin.lora_linear(None, buf[1:1 + 8 * 64].view(8, 64), W, None, 1.0)
    assert moin.device_status()["timeout_flag"] == 0
