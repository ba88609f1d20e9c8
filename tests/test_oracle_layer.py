"""Pins for the oracle's routed LoRA layer (Sec. 3.2: y = W x + W_b (W_a x); Sec. 3.3: one
expert per request; Sec. 4: no adapter => base model only).

Each test ties the oracle to something other than itself: a library fp64 matmul on the
merged weight, a closed form, an exact invariance, or a pure-Python brute force.  Shapes are
non-square and experts are mixed so that a transposed operand, a dropped term, a wrong sign
or a wrong slot index fails at least one of them.
"""
import os

import numpy as np
import pytest

import moin_inputs as mi
import oracle


def _case(T=37, d_in=48, d_out=80, E=5, r=8, seed=3, missing=()):
    rng = np.random.default_rng(seed)
    x = rng.normal(size=(T, d_in))
    W = rng.normal(size=(d_out, d_in)) * 0.1
    n_slots = E - len(missing)
    A = rng.normal(size=(n_slots, r, d_in)) * 0.1
    B = rng.normal(size=(n_slots, d_out, r)) * 0.1
    slot = np.full(E, -1, np.int32)
    kept = [e for e in range(E) if e not in missing]
    slot[kept] = np.arange(len(kept))
    te = rng.integers(0, E, size=T).astype(np.int32)
    return x, W, A, B, te, slot


def test_zero_B_is_base_layer():
    x, W, A, B, te, slot = _case()
    y = oracle.lora_linear(x, W, A, np.zeros_like(B), te, slot, 2.0)
    assert np.array_equal(y, oracle.lora_linear(x, W, None, None, None, None, 2.0))
    np.testing.assert_allclose(y, x @ W.T, rtol=0, atol=1e-12)


def test_single_expert_equals_merged_dense_weight():
    # LoRA merge identity: W x + s W_b W_a x = (W + s W_b W_a) x, via numpy's fp64 matmul.
    x, W, A, B, te, slot = _case()
    for e in range(5):
        y = oracle.lora_linear(x, W, A, B, np.full(x.shape[0], e, np.int32), slot, 1.7)
        merged = W + 1.7 * (B[slot[e]] @ A[slot[e]])
        np.testing.assert_allclose(y, x @ merged.T, rtol=0, atol=1e-12)


def test_mixed_experts_equal_per_group_merged_weight():
    x, W, A, B, te, slot = _case(T=64)
    y = oracle.lora_linear(x, W, A, B, te, slot, 2.0)
    for e in np.unique(te):
        rows = np.nonzero(te == e)[0]
        merged = W + 2.0 * (B[slot[e]] @ A[slot[e]])
        np.testing.assert_allclose(y[rows], x[rows] @ merged.T, rtol=0, atol=1e-12)


def test_rank_one_closed_form():
    # r = 1: y_tj = sum_i x_ti W_ji + s (a . x_t) b_j
    x, W, A, B, te, slot = _case(r=1)
    y = oracle.lora_linear(x, W, A, B, te, slot, 0.5)
    for t in range(x.shape[0]):
        a, b = A[slot[te[t]], 0], B[slot[te[t]], :, 0]
        np.testing.assert_allclose(y[t], W @ x[t] + 0.5 * np.dot(a, x[t]) * b, rtol=0, atol=1e-12)


def test_request_permutation_only_permutes_rows():
    # Experts never interact within a batch (abstract; Sec. 1): bitwise in the oracle.
    x, W, A, B, te, slot = _case(T=50)
    y = oracle.lora_linear(x, W, A, B, te, slot, 2.0)
    p = np.random.default_rng(9).permutation(50)
    yp = oracle.lora_linear(x[p], W, A, B, te[p], slot, 2.0)
    assert np.array_equal(yp, y[p])
    # any subset of the batch gives the same rows
    sub = p[:7]
    assert np.array_equal(oracle.lora_linear(x[sub], W, A, B, te[sub], slot, 2.0), y[sub])


def test_absent_adapter_falls_back_to_base():
    x, W, A, B, te, slot = _case(missing=(1, 3))
    te[:5] = [-1, 1, 3, 7, -9]   # no expert, two adapter-less topics, out of range ids
    y = oracle.lora_linear(x, W, A, B, te, slot, 2.0)
    base = x @ W.T
    for t in range(x.shape[0]):
        e = te[t]
        if e < 0 or e >= 5 or slot[e] < 0:
            np.testing.assert_allclose(y[t], base[t], rtol=0, atol=1e-12)
        else:
            assert np.abs(y[t] - base[t]).max() > 1e-3


def test_linear_in_scale():
    x, W, A, B, te, slot = _case()
    y0 = oracle.lora_linear(x, W, A, B, te, slot, 0.0)
    y1 = oracle.lora_linear(x, W, A, B, te, slot, 1.0)
    y4 = oracle.lora_linear(x, W, A, B, te, slot, 4.0)
    np.testing.assert_allclose(y0, x @ W.T, rtol=0, atol=1e-12)
    np.testing.assert_allclose(y4 - y0, 4.0 * (y1 - y0), rtol=0, atol=1e-11)


def test_brute_force_python_loops_tiny():
    x, W, A, B, te, slot = _case(T=5, d_in=6, d_out=4, E=3, r=2, seed=11)
    y = oracle.lora_linear(x, W, A, B, te, slot, 2.0)
    for t in range(5):
        s = slot[te[t]]
        for j in range(4):
            acc = sum(W[j][i] * x[t][i] for i in range(6))
            low = 0.0
            for p in range(2):
                low += B[s][j][p] * sum(A[s][p][i] * x[t][i] for i in range(6))
            assert abs(y[t][j] - (acc + 2.0 * low)) < 1e-13


def test_bf16_inputs_widen_exactly():
    case = mi.tiny_layer(seed=0)
    p = case.pool
    y_bits = oracle.lora_linear(mi.bf16_bits(case.x), mi.bf16_bits(case.W), mi.bf16_bits(p.A),
                                mi.bf16_bits(p.B), case.token_expert.numpy(), p.slot_of_expert.numpy(),
                                case.scale)
    y_f64 = oracle.lora_linear(mi.bf16_to_f64(case.x), mi.bf16_to_f64(case.W), mi.bf16_to_f64(p.A),
                               mi.bf16_to_f64(p.B), case.token_expert.numpy(), p.slot_of_expert.numpy(),
                               case.scale)
    assert np.array_equal(y_bits, y_f64)
    # the low-rank term must be visible at the tiny config's magnitudes
    base = mi.bf16_to_f64(case.x) @ mi.bf16_to_f64(case.W).T
    assert np.linalg.norm(y_f64 - base) / np.linalg.norm(y_f64) > 0.02


def test_round_bf16_matches_torch():
    import torch
    rng = np.random.default_rng(5)
    vals = np.concatenate([rng.normal(size=2000) * 10.0 ** rng.integers(-30, 30, size=2000),
                           [1.00390625, 1.01171875, -1.00390625, 0.0, 3.0e-40, 1e-45, 3.38e38, 3.4e38]])
    # torch rounds fp32 -> bf16 (RNE); use fp32-representable inputs so there is one rounding
    vals = vals.astype(np.float32).astype(np.float64)
    ref = torch.from_numpy(vals.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([oracle.round_bf16(v) for v in vals])
    assert np.array_equal(ref, got)


def test_golden_adapter_parameter_share():
    # Sec. 4: rank 128, token dim 2048; Sec. 1: the adapters are about 10 % of the model weights.
    path = os.path.join(os.path.dirname(__file__), "golden", "adapter_parameter_share.txt")
    vals = {}
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            k, v = line.split("=")
            vals[k.strip()] = float(v)
    per_rank = sum(d_in + d_out for _, d_in, d_out in mi.TINYLLAMA_PROJECTIONS)
    assert per_rank == int(vals["elements_per_rank_per_block"])
    total = int(vals["rank"]) * per_rank * int(vals["blocks"])
    assert total == int(vals["adapter_parameters"])
    share = total / vals["base_parameters"]
    assert abs(share - vals["paper_share"]) < 0.015


# ---------------------------------------------------------------------------------------------
# Variants from the paper's future-work list (Sec. 5): a rank per topic ("adaptive rank") and a function
# between the two low-rank matrices.  Same kind of pins as above.
# ---------------------------------------------------------------------------------------------
def test_per_slot_rank_equals_merged_weight_of_the_truncated_adapter():
    x, W, A, B, te, slot = _case(T=64, r=16)
    ranks = np.array([16, 8, 0, 12, 5], np.int32)          # slot -> rank (0: the adapter contributes nothing)
    y = oracle.lora_linear(x, W, A, B, te, slot, 2.0, slot_rank=ranks)
    for e in np.unique(te):
        rows = np.nonzero(te == e)[0]
        k = ranks[slot[e]]
        merged = W + 2.0 * (B[slot[e]][:, :k] @ A[slot[e]][:k, :])
        np.testing.assert_allclose(y[rows], x[rows] @ merged.T, rtol=0, atol=1e-12)
    # full rank for every slot = no rank table at all, bit for bit
    assert np.array_equal(oracle.lora_linear(x, W, A, B, te, slot, 2.0, slot_rank=np.full(5, 16, np.int32)),
                          oracle.lora_linear(x, W, A, B, te, slot, 2.0))
    # what is stored beyond a slot's rank is never read: poison it
    A2, B2 = A.copy(), B.copy()
    for s_, k in enumerate(ranks):
        A2[s_, k:, :] = np.nan
        B2[s_, :, k:] = np.inf
    assert np.array_equal(oracle.lora_linear(x, W, A2, B2, te, slot, 2.0, slot_rank=ranks), y)


@pytest.mark.parametrize("act,fn", [(oracle.ACT_RELU, lambda h: np.maximum(h, 0.0)),
                                    (oracle.ACT_SILU, lambda h: h / (1.0 + np.exp(-h))),
                                    (oracle.ACT_GELU, None)])
def test_activation_between_the_low_rank_matrices(act, fn):
    import math
    if fn is None:
        fn = np.vectorize(lambda v: 0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0))))
    x, W, A, B, te, slot = _case(T=50, missing=(3,))
    y = oracle.lora_linear(x, W, A, B, te, slot, 1.5, act=act)
    for t in range(x.shape[0]):
        ref = W @ x[t]
        if slot[te[t]] >= 0:
            ref = ref + 1.5 * (B[slot[te[t]]] @ fn(A[slot[te[t]]] @ x[t]))
        np.testing.assert_allclose(y[t], ref, rtol=0, atol=1e-12)
    # no activation = the paper's layer, bit for bit; and the activation does change routed rows only
    y0 = oracle.lora_linear(x, W, A, B, te, slot, 1.5)
    assert np.array_equal(oracle.lora_linear(x, W, A, B, te, slot, 1.5, act=oracle.ACT_NONE), y0)
    routed = slot[te] >= 0
    assert np.abs(y - y0)[routed].max() > 1e-3 and np.array_equal(y[~routed], y0[~routed])


def test_relu_rank_one_closed_form_and_rank_with_activation():
    # r = 1 with ReLU: the low-rank term is s * max(a . x, 0) * b - it vanishes exactly where a . x < 0
    x, W, A, B, te, slot = _case(r=1)
    y = oracle.lora_linear(x, W, A, B, te, slot, 0.5, act=oracle.ACT_RELU)
    base = oracle.lora_linear(x, W, None, None, None, None, 0.5)
    for t in range(x.shape[0]):
        a, b = A[slot[te[t]], 0], B[slot[te[t]], :, 0]
        np.testing.assert_allclose(y[t], base[t] + 0.5 * max(a @ x[t], 0.0) * b, rtol=0, atol=1e-12)
        if a @ x[t] < 0:
            assert np.array_equal(y[t], base[t])
    # rank table and activation together: SiLU is applied to the rows the slot has, the others are not read
    x, W, A, B, te, slot = _case(T=40, r=8)
    ranks = np.array([8, 3, 8, 1, 6], np.int32)
    y = oracle.lora_linear(x, W, A, B, te, slot, 2.0, slot_rank=ranks, act=oracle.ACT_SILU)
    for t in range(x.shape[0]):
        s_, k = slot[te[t]], ranks[slot[te[t]]]
        h = A[s_][:k] @ x[t]
        np.testing.assert_allclose(y[t], W @ x[t] + 2.0 * (B[s_][:, :k] @ (h / (1.0 + np.exp(-h)))), rtol=0, atol=1e-12)
