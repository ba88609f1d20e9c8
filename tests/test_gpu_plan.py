"""Batch plan (token bucketing) on the GPU against the oracle's stable grouping: integer work, bit-exact."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_09687_b200 as moin
from gpu_util import DEV

pytestmark = pytest.mark.gpu


def _check(te: np.ndarray, E: int):
    plan = moin.plan_build(torch.from_numpy(te).to(DEV), E, moin.PLAN_AUTO)
    got = plan.read()
    T = len(te)
    ident = np.arange(E, dtype=np.int32)  # plan groups by expert id: slot table = identity
    ref = oracle.bucket(te, ident, E)
    assert got["S"] == ref["S"]
    assert np.array_equal(got["perm"], ref["perm"])
    assert np.array_equal(got["seg_expert"], ref["seg_slot"])
    assert np.array_equal(got["seg_start"], ref["seg_start"])
    assert plan.c.n_segments == ref["S"]
    assert plan.c.n_lora_tokens == int(ref["seg_start"][-1])
    if ref["S"]:
        assert plan.c.max_segment == int(np.diff(ref["seg_start"]).max())
    # tiles: maximal runs of equal (sanitised) id, cut every 128 rows, covering [0, T) in order
    key = np.where((te >= 0) & (te < E), te, -1)
    row0, rows, tex = got["tile_row0"], got["tile_rows"], got["tile_expert"]
    assert rows.sum() == T and (rows >= 1).all() and (rows <= 128).all()
    assert np.array_equal(row0, np.concatenate([[0], np.cumsum(rows)[:-1]]))
    exp_tiles = 0
    start = 0
    for t in range(1, T + 1):
        if t == T or key[t] != key[start]:
            exp_tiles += -(-(t - start) // 128)
            start = t
    assert got["n_tiles"] == exp_tiles
    for a, n, e in zip(row0, rows, tex):
        assert (key[a:a + n] == e).all()
    return plan


def test_plan_decode_like():
    rng = np.random.default_rng(1)
    _check(rng.integers(0, 500, size=256).astype(np.int32), 500)


def test_plan_prefill_like_multi_chunk():
    rng = np.random.default_rng(2)
    req = rng.integers(0, 5000, size=32)
    plan = _check(np.repeat(req, 512).astype(np.int32), 5000)
    assert plan.mode == moin.PLAN_TILES


def test_plan_ragged_and_edge_cases():
    rng = np.random.default_rng(3)
    moin.device_status_reset()
    te = rng.integers(-1, 9, size=1000).astype(np.int32)
    te[[5, 77]] = [1234, -7]   # out of range ids: treated as "no expert" and counted
    _check(te, 8)
    assert moin.device_status()["invalid_expert_ids"] == 2 + int((te == 8).sum())
    _check(np.array([3], np.int32), 8)                       # one token
    _check(np.full(700, 2, np.int32), 8)                     # one expert
    _check(np.full(300, -1, np.int32), 8)                    # no expert at all
    _check(np.arange(300, dtype=np.int32), 300)              # all distinct
    lens = rng.integers(1, 33, size=16)
    _check(np.repeat(rng.integers(0, 8, size=16), lens).astype(np.int32), 8)   # ragged requests
    assert _check(rng.integers(0, 500, size=256).astype(np.int32), 500).mode == moin.PLAN_SEGMENTS


def test_plan_single_launch_and_chunked_paths_at_the_switch():
    # up to 1024 tokens: one single-CTA launch (shared-memory sort); beyond: the chunked launches
    rng = np.random.default_rng(7)
    for T, E in [(1024, 5000), (1025, 5000), (1023, 37), (200, 9000), (600, 70000), (33, 2), (31, 500), (513, 8)]:
        te = rng.integers(-1, E, size=T).astype(np.int32)
        te[rng.integers(0, T, size=T // 4)] = rng.integers(0, min(E, 6))   # a few long segments too
        _check(te, E)
    _check(np.repeat(rng.integers(0, 3, size=4), 256).astype(np.int32), 3)   # runs longer than one tile


def test_plan_all_distinct_at_every_sort_width():
    # T equal to the single-launch sort width with every token on its own expert: as many segments as the
    # sort has slots, so the end marker of the segment list sits one past the last sort slot
    for T in (128, 256, 512, 1024):
        for mode in (moin.PLAN_SEGMENTS, moin.PLAN_TILES):
            te = np.arange(T, dtype=np.int32)
            plan = moin.plan_build(torch.from_numpy(te).to(DEV), T, mode)
            got = plan.read()
            assert got["S"] == T
            assert np.array_equal(got["perm"], te) and np.array_equal(got["seg_expert"], te)
            assert np.array_equal(got["seg_start"], np.arange(T + 1))
            if mode == moin.PLAN_TILES:
                assert got["n_tiles"] == T and np.array_equal(got["tile_expert"], te)
        _check(np.arange(T, dtype=np.int32)[::-1].copy(), T)


def test_plan_is_deterministic():
    rng = np.random.default_rng(4)
    te = torch.from_numpy(rng.integers(0, 100, size=5000).astype(np.int32)).to(DEV)
    a = moin.plan_build(te, 100).read()
    b = moin.plan_build(te, 100).read()
    assert all(np.array_equal(a[k], b[k]) for k in ("perm", "seg_expert", "seg_start", "tile_row0"))
