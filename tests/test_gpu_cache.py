"""Two-tier adapter store on the GPU: experts' adapters in host memory, a few device slots, misses copied in
between the router and the layer.  The layer's output must not depend on what is resident: it is checked
against the oracle, which is given every expert's adapters.  The replacement policy (free slot first, else least
recently used among the slots the batch does not need) is checked against a model written here."""
import numpy as np
import pytest
import torch

import moin_inputs as mi
import oracle
import paper_2410_09687_b200 as moin
from gpu_util import DEV, assert_layer_close

pytestmark = pytest.mark.gpu


class _LruModel:
    def __init__(self, n_slots):
        self.expert_in = [-1] * n_slots
        self.last = [0] * n_slots
        self.tick = 0

    def admit(self, ids, E):
        self.tick += 1
        wanted = []
        for e in ids:
            if 0 <= e < E and e not in wanted:
                wanted.append(e)
        for e in wanted:
            if e in self.expert_in:
                self.last[self.expert_in.index(e)] = self.tick
        missed = 0
        for e in wanted:
            if e in self.expert_in:
                continue
            cand = [s for s in range(len(self.last)) if self.last[s] != self.tick]
            free = [s for s in cand if self.expert_in[s] < 0]
            v = free[0] if free else min(cand, key=lambda s: (self.last[s], s))
            self.expert_in[v], self.last[v] = e, self.tick
            missed += 1
        return missed


def test_layer_output_does_not_depend_on_residency_and_policy_is_lru():
    E, n_slots, r, d_in, d_out, T = 40, 12, 16, 256, 192, 96
    full = mi.make_pool(E, r, d_in, d_out, 41, 1)                # every expert's adapters (host)
    host = [(full.A.contiguous().pin_memory(), full.B.contiguous().pin_memory())]
    cache = moin.AdapterCache(host, n_slots, DEV)
    pool = cache.pools[0]
    model = _LruModel(n_slots)
    W = mi.normal_bf16((d_out, d_in), 0.02, 41, 2)
    rng = mi.np_rng(41, 3)
    ident = np.arange(E, dtype=np.int32)
    total_bytes = 0
    for step in range(8):
        hot = rng.choice(E, size=int(rng.integers(3, n_slots + 1)), replace=False)
        te = rng.choice(np.concatenate([hot, [-1]]), size=T).astype(np.int32)
        x = mi.normal_bf16((T, d_in), 1.0, 41, 10 + step)
        got = cache.admit(te)
        assert got["missed"] == model.admit(list(te), E), f"step {step}"
        assert got["bytes"] == got["missed"] * 2 * r * (d_in + d_out)
        total_bytes += got["bytes"]
        for e in range(E):                                       # host bookkeeping = the model's, slot by slot
            want = model.expert_in.index(e) if e in model.expert_in else -1
            assert cache.slot_of(e) == want
        plan = moin.plan_build(torch.from_numpy(te).to(DEV), E, moin.PLAN_SEGMENTS)
        y = moin.lora_linear(plan, x.to(DEV), W.to(DEV), pool, 2.0)
        torch.cuda.synchronize()
        ref = oracle.lora_linear(mi.bf16_bits(x), mi.bf16_bits(W), mi.bf16_bits(full.A), mi.bf16_bits(full.B), te, ident, 2.0)
        assert_layer_close(y, ref, f"cached layer, step {step}")
        assert np.array_equal(cache.table.cpu().numpy(),
                              np.array([model.expert_in.index(e) if e in model.expert_in else -1 for e in range(E)]))
    assert total_bytes > 0
    cache.close()


def test_a_batch_larger_than_the_cache_is_refused_and_changes_nothing():
    full = mi.make_pool(10, 8, 64, 64, 42, 1)
    cache = moin.AdapterCache([(full.A.contiguous().pin_memory(), full.B.contiguous().pin_memory())], 4, DEV)
    assert cache.admit([1, 2, 3])["missed"] == 3
    with pytest.raises(moin.MoinError, match="WORKSPACE"):
        cache.admit([0, 1, 2, 3, 4])
    assert [cache.slot_of(e) for e in (1, 2, 3, 0, 4)] == [0, 1, 2, -1, -1]
    assert cache.admit([3, 3, -1, 99, 1])["missed"] == 0          # repeats, "no adapter" and out-of-range ids
    cache.close()


def test_long_runs_through_the_cache():
    # the fused tensor-core path reads the same pools and table
    E, n_slots, r, d_in, d_out = 24, 6, 16, 512, 512
    full = mi.make_pool(E, r, d_in, d_out, 43, 1)
    cache = moin.AdapterCache([(full.A.contiguous().pin_memory(), full.B.contiguous().pin_memory())], n_slots, DEV)
    W = mi.normal_bf16((d_out, d_in), 0.02, 43, 2)
    ident = np.arange(E, dtype=np.int32)
    for step, req in enumerate(([3, 20, 7, 3], [11, 7, 0, 23], [5, 6, 9, 11])):
        te = np.repeat(np.array(req, np.int32), 160)
        x = mi.normal_bf16((len(te), d_in), 1.0, 43, 10 + step)
        cache.admit(req)
        plan = moin.plan_build(torch.from_numpy(te).to(DEV), E, moin.PLAN_TILES)
        y = moin.lora_linear(plan, x.to(DEV), W.to(DEV), cache.pools[0], 2.0)
        torch.cuda.synchronize()
        ref = oracle.lora_linear(mi.bf16_bits(x), mi.bf16_bits(W), mi.bf16_bits(full.A), mi.bf16_bits(full.B), te, ident, 2.0)
        assert_layer_close(y, ref, f"cached long runs, step {step}")
    cache.close()
