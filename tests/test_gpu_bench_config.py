"""The decode step exactly as bench.py times it - route, plan, four grouped projection calls, captured in a
CUDA graph and replayed - checked against the oracle: router ids for every request, layer outputs on a seeded
sample of tokens (each token's seven outputs are computed by the oracle one by one)."""
import os
import sys

import numpy as np
import pytest
import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench
import moin_inputs as mi
import oracle
import paper_2410_09687_b200 as moin
from gpu_util import DEV, ELEM_TOL, REL_FRO, assert_router_matches

pytestmark = pytest.mark.gpu


def test_decode_step_replayed_from_a_cuda_graph():
    wl = bench.LayerWorkload("decode", str(DEV))
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(3):
            wl.step(i)
        stream.synchronize()
        graphs = []
        for i in range(2):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                wl.step(i)
            graphs.append(g)
        for y in wl.y:
            y.zero_()
        graphs[1].replay()
        graphs[0].replay()          # batch 0 is the one left in the outputs
        graphs[0].replay()
        stream.synchronize()
    assert moin.device_status()["timeout_flag"] == 0
    # router: all 256 requests
    ref = oracle.route(mi.bf16_bits(wl.queries[0]), mi.bf16_bits(wl.router.centroids))
    ids = wl.req_expert.cpu().numpy()
    assert_router_matches(ids, ref)
    # layer: 24 sampled tokens x 7 projections, the oracle run on just those rows and their experts
    rows = np.sort(np.random.default_rng(5).choice(wl.T, size=24, replace=False))
    te = ids[rows]
    used = sorted(set(int(e) for e in te))
    remap = np.full(wl.E, -1, np.int32)
    remap[used] = np.arange(len(used))
    idx = torch.tensor(used, dtype=torch.long, device=DEV)
    rsel = torch.from_numpy(rows).to(DEV)
    for p, (name, d_in, d_out) in enumerate(wl.projs):
        want = oracle.lora_linear(mi.bf16_bits(wl.x[p][0][rsel]), mi.bf16_bits(wl.W[p]),
                                  mi.bf16_bits(wl.pools[p].A[idx]), mi.bf16_bits(wl.pools[p].B[idx]), te, remap, wl.scale)
        got = wl.y[p][rsel].double().cpu().numpy()
        err = np.linalg.norm(got - want) / np.linalg.norm(want)
        assert err <= REL_FRO, (name, err)
        assert (np.abs(got - want) <= ELEM_TOL * (1 + np.abs(want))).all(), name


def test_end_to_end_arm_delivers_the_step_results_to_the_host():
    """The pipelined end-to-end arm (packed pinned inputs -> copy-in stream -> kernels -> copy-out stream -> pinned
    results, several buffer sets in flight, replayed from a CUDA graph) must leave in host memory exactly what the
    plain step leaves on the device for the same batch."""
    wl = bench.LayerWorkload("decode", str(DEV))
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        wl.e2e_block(0)                       # eager once (also builds the buffer sets)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            wl.e2e_block(0)
        for lane in wl.lanes:
            lane["h_out"].zero_()
        g.replay()
        stream.synchronize()
    assert moin.device_status()["timeout_flag"] == 0
    # the last use of buffer set n inside block 0 is step k = E2E_BLOCK - E2E_LANES + n ... E2E_BLOCK - 1
    for k in range(wl.E2E_BLOCK - wl.E2E_LANES, wl.E2E_BLOCK):
        n, i = k % wl.E2E_LANES, k % bench.ROTATE
        wl.step(i)
        torch.cuda.synchronize()
        flat = wl.lanes[n]["h_out"]
        off = 0
        for p, y in enumerate(wl.y):
            nbytes = y.numel() * 2
            got = flat[off:off + nbytes].view(torch.bfloat16).view(y.shape)
            assert torch.equal(got, y.cpu()), (k, wl.projs[p][0])
            off += (nbytes + 255) // 256 * 256
