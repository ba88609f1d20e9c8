#!/usr/bin/env python
"""Benchmark of the MoIN serving hot path on B200 (one JSON line on stdout).

A "step" is one pass of the whole hot path over one batch of synthetic input:
  decode  (default): route 256 query embeddings over 500 centroids -> batch plan -> the seven
           TinyLlama-shaped projections with 500 rank-64 experts resident in HBM (256 single tokens)
  prefill: route 32 queries over 5 000 centroids -> plan -> seven projections, 32 x 512 tokens,
           5 000 rank-16 experts, Zipf(1.1) request experts
  router:  65 536 queries x 5 000 centroids x 768
  kmeans:  one Lloyd iteration of the topic clustering: 65 536 points x 5 000 centroids x 768 (assign with the
           router, group with the plan, update the centroids and their norms)
  forward: 22-block decoder, 64 x 256 tokens, 500 rank-64 experts on all seven projections

`value` is device-timed throughput with inputs resident in HBM; `e2e` repeats the measurement
with host buffers (pinned host -> device copies of the step's inputs and a device -> host copy of
its outputs inside the timed region).  `roofline` times the dominant kernel with CUDA events
inside the library; `cpu_baseline` times the CPU oracle on a bounded sample of the same work.
`--impl reference` times that oracle alone.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import moin_inputs as mi

NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS = 8000.0, 2250.0
FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS = 6650.0, 1590.0
ROTATE = 4  # distinct input batches rotated through the timed steps
GROUPS = [[0, 1, 2], [3], [4, 5], [6]]  # {q,k,v}, {o}, {gate,up}, {down}: independent inside a decoder block


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


# ----------------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc = None
        self.lines = []
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            sel = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            sel = str(device_index)
        self.cmd = ["nvidia-smi", "-i", sel, f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"]

    def start(self):
        try:
            self.proc = subprocess.Popen(self.cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no_samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------------------------
# workloads
# ----------------------------------------------------------------------------------------------
class LayerWorkload:
    """route -> plan -> seven projections.  decode: E=500 r=64 T=256; prefill: E=5000 r=16 32x512."""

    def __init__(self, kind: str, dev: str, grouped: bool = True, rank=None, cache_slots=None):
        import paper_2410_09687_b200 as moin
        self.moin, self.kind, self.dev, self.grouped = moin, kind, dev, grouped
        if kind == "decode":
            self.E, self.r, self.T, self.R, self.K, self.seed = 500, 64, 256, 256, 500, 1
            self.mode = moin.PLAN_SEGMENTS
        else:
            self.E, self.r, self.T, self.R, self.K, self.seed = 5000, 16, 16384, 32, 5000, 2
            self.mode = moin.PLAN_TILES
        if rank:   # side measurement at another rank (the paper trains its experts at 128, Sec. 4)
            self.r = int(rank)
        self.D, self.scale = 768, 2.0
        self.unit, self.units_per_step = "tokens", self.T
        self.projs = mi.TINYLLAMA_PROJECTIONS
        # resident state: centroid table, adapter pools, base weights
        rc = mi.planted_router(self.K, self.R * ROTATE, self.D, self.seed, device=dev)
        self.router = moin.Router(rc.centroids)
        self.queries = [rc.queries[i * self.R:(i + 1) * self.R].contiguous() for i in range(ROTATE)]
        self.labels = [rc.labels[i * self.R:(i + 1) * self.R] for i in range(ROTATE)]
        if kind == "prefill":   # Zipf-skewed request experts: planted labels -> skewed expert ids via the map
            cmaps = []
            for i in range(ROTATE):
                z = mi.zipf_experts(self.R, self.E, 1.1, self.seed, 21 + i)
                cmap = np.arange(self.K, dtype=np.int32)
                cmap[self.labels[i].cpu().numpy()] = z     # centroid of request j -> Zipf expert of request j
                cmaps.append(torch.from_numpy(cmap).to(dev))
            self.routers = [moin.Router(rc.centroids, m) for m in cmaps]
        else:
            self.routers = [self.router] * ROTATE
        self.pools, self.W, self.x, self.y = [], [], [], []
        self.cache = None
        if cache_slots:   # two-tier store: every expert's adapters in pinned host memory, cache_slots of them in HBM
            host = []
            for p, (name, d_in, d_out) in enumerate(self.projs):
                pool = mi.make_pool(self.E, self.r, d_in, d_out, self.seed, 30 + p)
                host.append((pool.A.contiguous().pin_memory(), pool.B.contiguous().pin_memory()))
            self.cache = moin.AdapterCache(host, int(cache_slots), dev)
            self.h_ids = torch.empty(self.R, dtype=torch.int32).pin_memory()
            self.cache_misses, self.cache_bytes, self.cache_steps = 0, 0, 0
        for p, (name, d_in, d_out) in enumerate(self.projs):
            if self.cache is not None:
                self.pools.append(self.cache.pools[p])
            else:
                pool = mi.make_pool(self.E, self.r, d_in, d_out, self.seed, 30 + p, device=dev)
                self.pools.append(moin.Pool(pool.A, pool.B, pool.slot_of_expert))
            self.W.append(mi.normal_bf16((d_out, d_in), 0.02, self.seed, 40 + p, 12, device=dev))
            self.x.append([mi.normal_bf16((self.T, d_in), 1.0, self.seed, 40 + p, 11, i, device=dev)
                           for i in range(ROTATE)])
            self.y.append(torch.empty(self.T, d_out, dtype=torch.bfloat16, device=dev))
        self.req_expert = torch.empty(self.R, dtype=torch.int32, device=dev)
        self.token_expert = torch.empty(self.T, dtype=torch.int32, device=dev)
        self.plan = moin.Plan(self.T, self.E, dev, self.mode)
        ws = max(moin.lib().moin_lora_linear_workspace_bytes(self.T, d_in, d_out, self.r) for _, d_in, d_out in self.projs)
        self.ws = torch.empty(ws, dtype=torch.uint8, device=dev)
        # projections that are independent inside a decoder block are issued as one grouped call
        self.groups = GROUPS if grouped else [[p] for p in range(len(self.projs))]
        self.jobgroups = [[moin.JobGroup([(self.x[p][i], self.W[p], self.pools[p], self.y[p]) for p in g])
                           for g in self.groups] for i in range(ROTATE)]
        self.ws = torch.empty(max(max(jg.workspace_bytes for jg in row) for row in self.jobgroups), dtype=torch.uint8,
                              device=dev)
        # host-side staging for the end-to-end arm
        self.n_host = ROTATE if kind == "decode" else 1
        self.h_q = [q.cpu().pin_memory() for q in self.queries[:self.n_host]]
        self.h_x = [[x.cpu().pin_memory() for x in xs[:self.n_host]] for xs in self.x]
        self.h_y = [torch.empty_like(y, device="cpu").pin_memory() for y in self.y]
        self.d_q = torch.empty_like(self.queries[0])
        self.d_x = [torch.empty_like(xs[0]) for xs in self.x]
        self.e2e_groups = [moin.JobGroup([(self.d_x[p], self.W[p], self.pools[p], self.y[p]) for p in g])
                           for g in self.groups]
        self.h2d = self.d_q.numel() * 2 + sum(x.numel() * 2 for x in self.d_x)
        self.d2h = sum(y.numel() * 2 for y in self.y)

    def _core(self, i: int, q, xs, jobgroups=None):
        moin = self.moin
        moin.route(self.routers[i], q, out_expert=self.req_expert)
        if self.cache is not None:   # the router's ids go to the host, the batch's missing adapters come in
            self.h_ids.copy_(self.req_expert, non_blocking=True)
            torch.cuda.current_stream().synchronize()
            got = self.cache.admit(self.h_ids.numpy())
            self.cache_misses += got["missed"]; self.cache_bytes += got["bytes"]; self.cache_steps += 1
        if self.kind == "decode":
            te = self.req_expert
        else:
            L = self.T // self.R   # plumbing: request id -> its tokens
            self.token_expert.view(self.R, L).copy_(self.req_expert.unsqueeze(1).expand(self.R, L))
            te = self.token_expert
        moin.plan_build(te, self.E, self.mode, plan=self.plan)
        for jg in jobgroups:
            moin.lora_linear_group(self.plan, jg, self.scale, workspace=self.ws)

    def step(self, i: int):
        i %= ROTATE
        self._core(i, self.queries[i], [xs[i] for xs in self.x], self.jobgroups[i])

    def step_e2e(self, i: int):
        i %= ROTATE
        j = i % self.n_host
        self.d_q.copy_(self.h_q[j], non_blocking=True)
        for p in range(len(self.projs)):
            self.d_x[p].copy_(self.h_x[p][j], non_blocking=True)
        self._core(i, self.d_q, self.d_x, self.e2e_groups)
        for p in range(len(self.projs)):
            self.h_y[p].copy_(self.y[p], non_blocking=True)

    # ---- end-to-end arm, pipelined: one stream copies inputs in, one runs the kernels, one copies results out; a
    # few buffer sets (device inputs, outputs, plan, workspace, pinned result buffers) rotate through them, so the
    # host <-> device copies of a step run beside the kernels of its neighbours while the kernels of different
    # steps never share the GPU
    E2E_BLOCK = 48  # steps issued per call of e2e_block (one CUDA graph holds that many)
    E2E_LANES = 3   # buffer sets

    @staticmethod
    def _packed(like, device, pin=False):
        """One flat byte buffer holding tensors shaped like `like` at 256-byte offsets, and the views into it."""
        offs, total = [], 0
        for t in like:
            offs.append(total)
            total += (t.numel() * t.element_size() + 255) // 256 * 256
        flat = torch.empty(total, dtype=torch.uint8, device=device)
        if pin:
            flat = flat.pin_memory()
        views = [flat[o:o + t.numel() * t.element_size()].view(t.dtype).view(t.shape) for o, t in zip(offs, like)]
        return flat, views

    def _make_lanes(self):
        moin, dev = self.moin, self.dev
        lanes = []
        ins = [self.queries[0]] + [xs[0] for xs in self.x]
        # a step's inputs (and its results) travel as ONE copy each way: host-side they sit packed in one pinned buffer
        self.h_in = []
        for j in range(self.n_host):
            flat, views = self._packed(ins, "cpu", pin=True)
            views[0].copy_(self.h_q[j])
            for p in range(len(self.projs)):
                views[1 + p].copy_(self.h_x[p][j])
            self.h_in.append(flat)
        for k in range(self.E2E_LANES):
            d_in, in_views = self._packed(ins, dev)
            d_out, y = self._packed(self.y, dev)
            d_q, d_x = in_views[0], in_views[1:]
            lanes.append({
                "d_q": d_q, "d_x": d_x, "y": y, "d_in": d_in, "d_out": d_out,
                "h_out": torch.empty(d_out.numel(), dtype=torch.uint8).pin_memory(),
                "req_expert": torch.empty(self.R, dtype=torch.int32, device=dev),
                "plan": moin.Plan(self.T, self.E, dev, self.mode),
                "ws": torch.empty_like(self.ws),
                "groups": [moin.JobGroup([(d_x[p], self.W[p], self.pools[p], y[p]) for p in g]) for g in self.groups]})
        self.e2e_streams = [torch.cuda.Stream() for _ in range(3)]   # copy in, kernels, copy out
        self.h2d, self.d2h = lanes[0]["d_in"].numel(), lanes[0]["d_out"].numel()
        return lanes

    def e2e_block(self, b: int):
        """E2E_BLOCK consecutive end-to-end steps (decode only); called on the timing stream."""
        if not hasattr(self, "lanes"):
            self.lanes = self._make_lanes()
        moin = self.moin
        origin = torch.cuda.current_stream()
        s_in, s_run, s_out = self.e2e_streams
        for st in self.e2e_streams:
            st.wait_stream(origin)
        # per buffer set: events of its last use inside this block (the block's ends are full joins)
        ran = [None] * self.E2E_LANES     # kernels done: the device inputs may be overwritten
        out = [None] * self.E2E_LANES     # results copied out: the device outputs may be overwritten
        for k in range(self.E2E_BLOCK):
            step = b * self.E2E_BLOCK + k
            n = step % self.E2E_LANES
            i, lane = step % ROTATE, self.lanes[n]
            j = i % self.n_host
            with torch.cuda.stream(s_in):
                if ran[n] is not None:
                    s_in.wait_event(ran[n])
                lane["d_in"].copy_(self.h_in[j], non_blocking=True)
                ready = torch.cuda.Event()
                ready.record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(ready)
                if out[n] is not None:
                    s_run.wait_event(out[n])
                moin.route(self.routers[i], lane["d_q"], out_expert=lane["req_expert"])
                moin.plan_build(lane["req_expert"], self.E, self.mode, plan=lane["plan"])
                for jg in lane["groups"]:
                    moin.lora_linear_group(lane["plan"], jg, self.scale, workspace=lane["ws"])
                ran[n] = torch.cuda.Event()
                ran[n].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ran[n])
                lane["h_out"].copy_(lane["d_out"], non_blocking=True)
                out[n] = torch.cuda.Event()
                out[n].record(s_out)
        for st in self.e2e_streams:
            origin.wait_stream(st)

    def distinct(self) -> float:
        vals = []
        for i in range(ROTATE):
            self.moin.route(self.routers[i], self.queries[i], out_expert=self.req_expert)
            vals.append(int(torch.unique(self.req_expert[self.req_expert >= 0]).numel()))
        return float(np.mean(vals))

    def algorithmic(self, n_distinct: float) -> dict:
        """Bytes / flops one step must move or compute: x, W, y once; every distinct adapter once."""
        T, r = self.T, self.r
        per = {"gemm": 0.0, "shrink": 0.0, "expand": 0.0}
        flops = 0.0
        for _, d_in, d_out in self.projs:
            per["gemm"] += d_out * d_in * 2 + T * d_in * 2 + T * d_out * 2
            per["shrink"] += n_distinct * r * d_in * 2 + T * d_in * 2 + T * r * 4
            per["expand"] += n_distinct * d_out * r * 2 + T * r * 4 + T * d_out * 2
            flops += 2.0 * T * d_in * d_out + 2.0 * T * r * (d_in + d_out)
        step_bytes = sum((d_out * d_in + T * d_in + T * d_out + n_distinct * r * (d_in + d_out)) * 2
                         for _, d_in, d_out in self.projs) + self.R * self.D * 2 + self.K * self.D * 2
        # long-run mode: the fused GEMM's own work is the base product plus hi and lo K blocks of the rank
        rb = (r + 63) // 64 * 64
        fused = sum(2.0 * T * d_out * (d_in + 2 * rb) for _, d_in, d_out in self.projs)
        shrink_tc = sum(2.0 * T * r * d_in for _, d_in, d_out in self.projs)
        return {"per_kernel_bytes": per, "step_bytes": step_bytes, "step_flops": flops,
                "per_kernel_flops": {"lora_fused_tc": fused, "lora_shrink_tc": shrink_tc}}

    def config(self) -> dict:
        name = (f"decode: 7 TinyLlama projections, 500 experts rank {self.r}, 256 single tokens, router 256x500x768"
                if self.kind == "decode" else
                f"prefill: 7 TinyLlama projections, 5000 experts rank {self.r}, 32x512 tokens Zipf(1.1), router 32x5000x768")
        return {"workload": name, "calls": ("grouped {q,k,v} {o} {gate,up} {down}" if self.grouped else "one call per projection"),
                "tokens_per_step": self.T, "experts": self.E, "rank": self.r, "lora_scale": self.scale,
                "l2": f"inputs rotate over {ROTATE} batches; per-step working set exceeds L2"}

    def oracle_sample(self, n_tokens: int) -> float:
        """Seconds the CPU oracle needs for route + the seven projections of n_tokens tokens: the first tokens of
        batch 0, then of batch 1, ... (a sample larger than one batch goes round the rotating batches)."""
        import oracle
        total, done, b = 0.0, 0, 0
        while done < n_tokens:
            n = min(self.T, n_tokens - done)
            total += self._oracle_batch(oracle, b % ROTATE, n)
            done += n
            b += 1
        return total

    def _oracle_batch(self, oracle, b: int, n_tokens: int) -> float:
        n_req = max(1, n_tokens * self.R // self.T)
        rows = np.arange(n_tokens)
        q = mi.bf16_bits(self.queries[b][:n_req])
        c = mi.bf16_bits(self.router.centroids)
        self.step(b)
        torch.cuda.synchronize()
        te = (self.req_expert if self.kind == "decode" else self.token_expert).cpu().numpy()[rows]
        used = sorted(set(int(e) for e in te if e >= 0))
        remap = np.full(self.E, -1, np.int32)
        remap[used] = np.arange(len(used))
        idx = torch.tensor(used, dtype=torch.long, device=self.dev)
        host = []
        for p, (_, d_in, d_out) in enumerate(self.projs):
            host.append((mi.bf16_bits(self.x[p][b][:n_tokens]), mi.bf16_bits(self.W[p]),
                         mi.bf16_bits(self.pools[p].A[idx]), mi.bf16_bits(self.pools[p].B[idx])))
        t0 = time.perf_counter()
        oracle.route(q, c)
        for x, W, A, B in host:
            oracle.lora_linear(x, W, A, B, te, remap, self.scale)
        return time.perf_counter() - t0


class RouterWorkload:
    def __init__(self, dev: str, Q: int = 65536, K: int = 5000, D: int = 768):
        import paper_2410_09687_b200 as moin
        self.moin, self.dev, self.Q, self.K, self.D = moin, dev, Q, K, D
        rc = mi.planted_router(K, Q, D, 3, device=dev)
        self.router = moin.Router(rc.centroids)
        # rotate by rolling the query matrix: same multiset of queries, different rows per buffer
        self.queries = [rc.queries] + [torch.roll(rc.queries, shifts=i * 4099, dims=0).contiguous() for i in range(1, ROTATE)]
        self.out = torch.empty(Q, dtype=torch.int32, device=dev)
        self.unit, self.units_per_step = "queries", Q
        self.h_q = [self.queries[0].cpu().pin_memory()]
        self.h_out = torch.empty(Q, dtype=torch.int32).pin_memory()
        self.d_q = torch.empty_like(rc.queries)
        self.h2d, self.d2h = Q * D * 2, Q * 4

    def step(self, i: int):
        self.moin.route(self.router, self.queries[i % ROTATE], out_expert=self.out)

    def step_e2e(self, i: int):
        self.d_q.copy_(self.h_q[0], non_blocking=True)
        self.moin.route(self.router, self.d_q, out_expert=self.out)
        self.h_out.copy_(self.out, non_blocking=True)

    def config(self) -> dict:
        return {"workload": f"router stress: {self.Q} queries x {self.K} centroids x {self.D}, planted clusters",
                "l2": f"query matrix (100.7 MB) rotates over {ROTATE} buffers (> L2 in total)"}

    def algorithmic(self) -> dict:
        return {"flops": 2.0 * self.Q * self.K * self.D, "bytes": (self.Q + self.K) * self.D * 2 + self.Q * 4}

    def oracle_sample(self, n: int) -> float:
        import oracle
        q = mi.bf16_bits(self.queries[0][:n])
        c = mi.bf16_bits(self.router.centroids)
        t0 = time.perf_counter()
        oracle.route(q, c)
        return time.perf_counter() - t0


class KMeansWorkload:
    """One K-means (Lloyd) iteration over the router-stress data: assign, group, update (in place)."""

    def __init__(self, dev: str, N: int = 65536, K: int = 5000, D: int = 768):
        import paper_2410_09687_b200 as moin
        self.moin, self.dev, self.N, self.K, self.D = moin, dev, N, K, D
        rc = mi.planted_router(K, N, D, 3, device=dev)
        g = torch.Generator(device=dev).manual_seed(7)
        start = (rc.centroids.float() + 0.4 * torch.randn(K, D, generator=g, device=dev) / D ** 0.5).to(torch.bfloat16)
        self.start = start
        self.cent = start.clone()                  # updated in place every step
        self.router = moin.Router(self.cent)       # borrows self.cent and owns the inverse norms
        self.points = [rc.queries] + [torch.roll(rc.queries, shifts=i * 4099, dims=0).contiguous() for i in range(1, ROTATE)]
        self.assign = torch.empty(N, dtype=torch.int32, device=dev)
        self.plan = moin.Plan(N, K, dev, moin.PLAN_SEGMENTS)
        self.router.workspace(N)
        self.unit, self.units_per_step = "points", N
        self.h_x = [self.points[0].cpu().pin_memory()]
        self.h_c = torch.empty(K, D, dtype=torch.bfloat16).pin_memory()
        self.d_x = torch.empty_like(rc.queries)
        self.h2d, self.d2h = N * D * 2, K * D * 2

    def _iterate(self, x):
        moin = self.moin
        moin.route(self.router, x, out_expert=self.assign)
        moin.plan_build(self.assign, self.K, moin.PLAN_SEGMENTS, plan=self.plan)
        moin.kmeans_update(self.plan, x, self.cent, centroids_new=self.cent, inv_norm_new=self.router.inv_norm)

    def step(self, i: int):
        self._iterate(self.points[i % ROTATE])

    def step_e2e(self, i: int):
        self.d_x.copy_(self.h_x[0], non_blocking=True)
        self._iterate(self.d_x)
        self.h_c.copy_(self.cent, non_blocking=True)

    def config(self) -> dict:
        return {"workload": f"k-means iteration: {self.N} points x {self.K} centroids x {self.D}, planted clusters, "
                            f"perturbed start; assign (router) + group (plan) + update",
                "l2": f"point matrix (100.7 MB) rotates over {ROTATE} buffers (> L2 in total)"}

    def algorithmic(self) -> dict:
        return {"flops": 2.0 * self.N * self.K * self.D,
                "bytes": (self.N + 2 * self.K) * self.D * 2 + self.N * 4,
                "update_bytes": (self.N + self.K) * self.D * 2 + self.N * 4}

    def oracle_sample(self, n: int) -> float:
        import oracle
        x = mi.bf16_bits(self.points[0][:n])
        c = mi.bf16_bits(self.start)
        t0 = time.perf_counter()
        a = oracle.route(x, c)["centroid"]
        oracle.kmeans_update(x, c, a)
        return time.perf_counter() - t0


class ForwardWorkload:
    """22-block decoder, 64 x 256 tokens, 500 rank-64 experts on all 7 projections (pool ~50 GB)."""

    def __init__(self, dev: str, n_layers: int = 22, R: int = 64, L: int = 256):
        import paper_2410_09687_b200 as moin
        self.moin, self.dev = moin, dev
        cfg = mi.DecoderConfig(n_layers=n_layers)
        self.cfg, self.R, self.L, self.T = cfg, R, L, R * L
        model = mi.decoder_model(cfg, seed=4, device=dev)
        order = ("q", "k", "v", "o", "gate", "up", "down")
        pools = [{p: moin.Pool(model.pools[l][p].A, model.pools[l][p].B, model.pools[l][p].slot_of_expert)
                  for p in order} for l in range(n_layers)]
        self.gm = moin.DecoderModel(cfg, model.embed, model.lm_head, model.final_norm, model.attn_norm, model.mlp_norm,
                                    [{p: model.W[l][p] for p in order} for l in range(n_layers)], pools, cfg.E, cfg.scale)
        self.batches = [mi.decoder_batch(cfg, [L] * R, seed=4 + i, device=dev) for i in range(ROTATE)]
        self.logits = torch.empty(self.T, cfg.vocab, dtype=torch.bfloat16, device=dev)
        self.unit, self.units_per_step = "tokens", self.T
        self.h_tok = [b.tokens.cpu().pin_memory() for b in self.batches]
        self.d_tok = torch.empty_like(self.batches[0].tokens)
        self.h_last = torch.empty(R, cfg.vocab, dtype=torch.bfloat16).pin_memory()
        self.last = torch.empty(R, cfg.vocab, dtype=torch.bfloat16, device=dev)
        self.h2d, self.d2h = self.T * 4, R * cfg.vocab * 2
        self.gm.workspace(R, self.T)

    def step(self, i: int):
        b = self.batches[i % ROTATE]
        self.moin.decoder_forward(self.gm, b.tokens, b.cu_seqlens, b.req_expert, self.L, logits=self.logits)

    def step_e2e(self, i: int):
        b = self.batches[i % ROTATE]
        self.d_tok.copy_(self.h_tok[i % ROTATE], non_blocking=True)
        self.moin.decoder_forward(self.gm, self.d_tok, b.cu_seqlens, b.req_expert, self.L,
                                  logits_mode=self.moin.LOGITS_LAST, logits=self.last)
        self.h_last.copy_(self.last, non_blocking=True)

    def config(self) -> dict:
        return {"workload": f"full decoder forward: {self.cfg.n_layers} TinyLlama-shaped blocks, {self.R}x{self.L} tokens, "
                            f"500 experts rank 64 on 7 projections, all-position logits",
                "l2": "activations and weights per step far exceed L2"}

    def algorithmic(self) -> dict:
        c, T = self.cfg, self.T
        per_layer = sum(2.0 * T * d_in * d_out + 2.0 * T * c.r * (d_in + d_out) for _, d_in, d_out in c.projections())
        attn = 2.0 * 2.0 * self.R * c.n_heads * (self.L * (self.L + 1) / 2) * c.head_dim
        return {"flops": c.n_layers * (per_layer + attn) + 2.0 * T * c.hidden * c.vocab}


# ----------------------------------------------------------------------------------------------
# measurement helpers
# ----------------------------------------------------------------------------------------------
def dist_setup(n_gpus: int, backend: str = "nccl"):
    """One process per GPU (replicas): reads RANK / LOCAL_RANK / WORLD_SIZE; the process group only carries the
    barrier and the max-over-ranks of the timing.  `backend="gloo"` runs the same logic on CPU (tests)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        if backend == "nccl":
            torch.cuda.set_device(local)
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(backend)
    elif backend == "nccl":
        torch.cuda.set_device(0)
        local = 0
    return world, rank, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(world, v: float) -> float:
    if world > 1:
        import torch.distributed as dist
        dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
        t = torch.tensor([v], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())
    return v


def whole_job_value(world: int, units_per_step: float, ms_per_step_max: float) -> float:
    """Aggregate throughput of `world` replicas that each process units_per_step per step (weak scaling):
    all the units divided by the slowest rank's time."""
    return world * units_per_step / (ms_per_step_max * 1e-3)


def timed_loop(world, fn, steps: int, warmup: int, use_graph: bool) -> float:
    """ms per step over exactly `steps` steps, CUDA events on the launching stream, barrier + sync both sides."""
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(max(warmup, 3)):
            fn(i)
        stream.synchronize()
        graphs = None
        if use_graph:
            try:
                graphs = []
                for i in range(ROTATE):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=stream):
                        fn(i)
                    graphs.append(g)
                for g in graphs:
                    g.replay()
                stream.synchronize()
            except Exception as e:  # pragma: no cover
                sys.stderr.write(f"[bench] CUDA graph capture failed ({e}); timing plain launches\n")
                graphs = None
                torch.cuda.synchronize()
        barrier(world)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        if graphs is not None:
            for i in range(steps):
                graphs[i % ROTATE].replay()
        else:
            for i in range(steps):
                fn(i)
        e1.record(stream)
        stream.synchronize()
        barrier(world)
        torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps, graphs is not None


def wl_cache_free(wl) -> bool:
    return getattr(wl, "cache", None) is None


def profile_pass(moin, fn, steps: int):
    """Per-kernel device time (CUDA events inside the library, on the launching stream)."""
    moin.profile_enable(65536)
    try:
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            fn(0)
            stream.synchronize()
            moin.profile_read()
            for i in range(steps):
                fn(i)
            stream.synchronize()
        recs = moin.profile_read()
    finally:
        moin.profile_enable(0)
    agg = {}
    for r in recs:
        a = agg.setdefault(r["kernel"], {"launches": 0, "brackets": 0, "ms": 0.0})
        a["launches"] += r["launches"]; a["brackets"] += 1; a["ms"] += r["ms"]
    launches_per_step = sum(a["launches"] for a in agg.values()) / steps
    return agg, launches_per_step


def kernel_timeline(fn, use_graph: bool, steps: int = 6):
    """Start / end of every kernel of one step, from the profiler's activity records of `steps` replays (the
    kernels keep running concurrently while they are recorded).  Returns (rows, span_us) for the median-length
    step: rows = [(name, start_us, end_us)] relative to the step's first kernel.  None if no records come back."""
    try:
        from torch.profiler import ProfilerActivity, profile
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            graphs = []
            for i in range(ROTATE):
                fn(i)
            stream.synchronize()
            if use_graph:
                for i in range(ROTATE):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=stream):
                        fn(i)
                    graphs.append(g)
            run = (lambda i: graphs[i % ROTATE].replay()) if use_graph else fn
            for i in range(ROTATE):
                run(i)
            stream.synchronize()
            with profile(activities=[ProfilerActivity.CUDA]) as prof:
                for i in range(steps + 1):
                    run(i)
                stream.synchronize()
        evs = sorted((e for e in prof.events() if e.device_type == torch.autograd.DeviceType.CUDA and "moin::" in e.name),
                     key=lambda e: e.time_range.start)
        if not evs:
            return None
        first = evs[0].name
        cuts = [i for i, e in enumerate(evs) if e.name == first]
        if len(cuts) < 3:
            return None
        spans = [(evs[cuts[k + 1]].time_range.start - evs[cuts[k]].time_range.start, k) for k in range(len(cuts) - 1)]
        span, k = sorted(spans)[len(spans) // 2]
        t0 = evs[cuts[k]].time_range.start
        rows = [(e.name, e.time_range.start - t0, e.time_range.end - t0) for e in evs[cuts[k]:cuts[k + 1]]]
        return rows, span
    except Exception as e:  # pragma: no cover
        sys.stderr.write(f"[bench] no kernel timeline ({e})\n")
        return None


def critical_path(rows, span_us: float) -> dict:
    """Where a step's time goes, from its kernel timeline.  Kernels on the call's own stream follow one another, so
    their durations add up; the base GEMMs of the short-segment path run on side streams beside the shrink, and
    only the part of a GEMM that outlasts the shrink it runs beside delays the expand ("gemm_exposed").  The
    remainder of the step is launch gaps.  No entry can exceed the step."""
    def short(n):
        n = n.split("moin::")[1].split("(")[0].split("<")[0]
        return n.replace("_kernel", "")
    main, side = {}, []
    ordered = sorted(rows, key=lambda r: r[1])
    for name, a, b in ordered:
        k = short(name)
        if k.startswith("tc_gemm") or k.startswith("gemm_warp"):
            side.append((a, b))
        else:
            main[k] = main.get(k, 0.0) + (b - a)
    exposed = 0.0
    if side and any(k.startswith("lora_expand") for k in main):
        # per expand launch: how long after the end of the shrink before it did the last GEMM before it end?
        exp = [(a, b) for n, a, b in ordered if "lora_expand" in n]
        shr = [(a, b) for n, a, b in ordered if "lora_shrink" in n]
        for (ea, _), (_, sb) in zip(exp, shr):
            g_end = max([b for a, b in side if a < ea] or [0.0])
            exposed += max(0.0, min(g_end, ea) - sb)
        out = dict(main)
        out["gemm_exposed"] = exposed
    else:   # everything on one stream
        out = dict(main)
        for a, b in side:
            out["tc_gemm"] = out.get("tc_gemm", 0.0) + (b - a)
    out = {k: round(v, 2) for k, v in out.items()}
    out["gaps"] = round(max(0.0, span_us - sum(out.values())), 2)
    out["step_us"] = round(span_us, 2)
    return out


def tensor_roofline(top: str, a: dict, alg: dict, prof_steps: int, peaks: dict, kind: str) -> dict:
    """Roofline object of a long-run tensor-core kernel: ITS OWN flops per launch over its own launch time
    (CUDA-event brackets, the kernel alone between them), against the burst peak a kernel timed in isolation sees."""
    fl = alg["per_kernel_flops"][top] * prof_steps / a["launches"]
    sec = a["ms"] * 1e-3 / a["launches"]
    ach = fl / sec / 1e12
    return {"kernel": top, "bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
            "frac": ach / peaks["bf16_tflops"], "frac_sustained": ach / peaks["bf16_tflops_sustained"],
            "frac_nominal": ach / NOMINAL_BF16_TFLOPS, "peak_source": peaks["source"] + " (burst)",
            "algorithmic_flops_per_launch": fl, "avg_launch_ms": sec * 1e3, "traffic": traffic_for(top, kind)}


def side_prefill(moin, dev: str, peaks: dict, local: int) -> dict:
    """Prefill workload (32 x 512 tokens, 5000 rank-16 experts) as an extra key of the default line."""
    wl = LayerWorkload("prefill", dev)
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    ms, graphed = timed_loop(1, wl.step, 400, 5, True)     # >= 0.5 s of timed work
    clocks = sampler.stop()
    agg, _ = profile_pass(moin, wl.step, 10)
    nd = wl.distinct()
    alg = wl.algorithmic(nd)
    t_tc = alg["step_flops"] / (peaks["bf16_tflops"] * 1e12)
    t_hbm = alg["step_bytes"] / (peaks["hbm_gbs"] * 1e9)
    out = {"workload": wl.config()["workload"], "ms_per_step": ms, "tokens_per_s": wl.T / (ms * 1e-3),
           "launch": "cuda_graph replay" if graphed else "plain launches", "clocks": clocks,
           "step_roofline": {"bound": "tensor" if t_tc >= t_hbm else "hbm", "roofline_ms": max(t_tc, t_hbm) * 1e3,
                             "frac": max(t_tc, t_hbm) * 1e3 / ms,
                             "frac_nominal": max(alg["step_flops"] / (NOMINAL_BF16_TFLOPS * 1e12),
                                                 alg["step_bytes"] / (NOMINAL_HBM_GBS * 1e9)) * 1e3 / ms,
                             "peak": "burst"},
           "distinct_experts": nd}
    if "lora_fused_tc" in agg:
        out["roofline"] = tensor_roofline("lora_fused_tc", agg["lora_fused_tc"], alg, 10, peaks, "prefill")
    out["kernels"] = {k: {"launches": a["launches"], "ms_per_launch": a["ms"] / max(a["launches"], 1)} for k, a in agg.items()}
    del wl
    torch.cuda.empty_cache()
    return out


def side_forward(moin, dev: str, peaks: dict, local: int) -> dict:
    """Full decoder forward (22 blocks, 64 x 256 tokens, 500 rank-64 experts) as an extra key of the default line."""
    wl = ForwardWorkload(dev)
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    ms, _ = timed_loop(1, wl.step, 14, 3, False)           # >= 0.5 s of timed work
    clocks = sampler.stop()
    alg = wl.algorithmic()
    ach = alg["flops"] / (ms * 1e-3) / 1e12
    out = {"workload": wl.config()["workload"], "ms_per_step": ms, "tokens_per_s": wl.T / (ms * 1e-3), "clocks": clocks,
           "achieved_tflops": ach, "frac": ach / peaks["bf16_tflops_sustained"], "peak": "sustained",
           "frac_burst": ach / peaks["bf16_tflops"], "frac_nominal": ach / NOMINAL_BF16_TFLOPS,
           "algorithmic_flops": alg["flops"]}
    del wl
    torch.cuda.empty_cache()
    return out


def traffic_for(kernel: str, workload: str):
    """DRAM bytes per launch from the committed ncu capture, or None when the kernel source changed since."""
    p = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(p):
        return None
    try:
        d = json.load(open(p)).get(f"{kernel}:{workload}")
        if not d:
            return None
        src = os.path.join(ROOT, d["source"])
        if hashlib.sha256(open(src, "rb").read()).hexdigest()[:16] != d["source_sha256_16"]:
            return None
        return d["dram_bytes_per_launch"]
    except Exception:
        return None


def adaptive_oracle(sample_fn, first: int, cap: int, target_s: float = 20.0):
    """Times the oracle on `first` units, then once more on a sample sized from that rate for target_s seconds
    (small samples run slower per unit, so the second run ends up around half of target_s)."""
    t = sample_fn(first)
    n = int(min(cap, max(first, first * target_s / max(t, 1e-3))))
    if n > first * 1.5:
        t = sample_fn(n)
    else:
        n = first
    return n, t


# ----------------------------------------------------------------------------------------------
def run_reference(args):
    """Reference arm = the CPU oracle as it stands, on this machine's host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    oracle.build()
    cores = oracle.num_threads()
    kind = args.workload
    rng_seed = {"decode": 1, "prefill": 2, "router": 3, "forward": 4, "kmeans": 3}[kind]
    if kind in ("router", "kmeans"):
        n, K, D = 256, 5000, 768
        rc = mi.planted_router(K, n, D, rng_seed)
        q, c = mi.bf16_bits(rc.queries), mi.bf16_bits(rc.centroids)
        if kind == "router":
            fn = lambda: oracle.route(q, c)
            unit, metric, sample = "queries/s", "router_queries_per_s", f"{n} of 65536 queries per step, all 5000 centroids"
            cfgname = "router stress: 65536 queries x 5000 centroids x 768, planted clusters"
        else:
            fn = lambda: oracle.kmeans_update(q, c, oracle.route(q, c)["centroid"])
            unit, metric, sample = "points/s", "kmeans_points_per_s", f"assign + update of {n} of 65536 points per step, all 5000 centroids"
            cfgname = "k-means iteration: 65536 points x 5000 centroids x 768, planted clusters"
    else:
        if kind == "forward":
            sys.stderr.write("[bench] reference arm for 'forward' times the seven projections of one block\n")
        E, r, n = (500, 64, 32) if kind != "prefill" else (5000, 16, 32)
        te = np.random.default_rng(rng_seed).integers(0, 8, size=n).astype(np.int32)
        slot = np.full(E, -1, np.int32); slot[:8] = np.arange(8)
        host = []
        for p, (_, d_in, d_out) in enumerate(mi.TINYLLAMA_PROJECTIONS):
            pool = mi.make_pool(8, r, d_in, d_out, rng_seed, 30 + p)
            host.append((mi.bf16_bits(mi.normal_bf16((n, d_in), 1.0, rng_seed, 40 + p, 11)),
                         mi.bf16_bits(mi.normal_bf16((d_out, d_in), 0.02, rng_seed, 40 + p, 12)),
                         mi.bf16_bits(pool.A), mi.bf16_bits(pool.B)))
        rc = mi.planted_router(500 if kind != "prefill" else 5000, n if kind == "decode" else 1, 768, rng_seed)
        q, c = mi.bf16_bits(rc.queries), mi.bf16_bits(rc.centroids)

        def fn():
            oracle.route(q, c)
            for x, W, A, B in host:
                oracle.lora_linear(x, W, A, B, te, slot, 2.0)
        unit, metric = "tokens/s", "routed_lora_tokens_per_s"
        sample = f"{n} tokens per step through route + the 7 projections (8 distinct adapters)"
        cfgname = {"decode": "decode: 7 TinyLlama projections, 500 experts rank 64, 256 single tokens, router 256x500x768",
                   "prefill": "prefill: 7 TinyLlama projections, 5000 experts rank 16, 32x512 tokens Zipf(1.1), router 32x5000x768",
                   "forward": "full decoder forward (projections of one block as the sample)"}[kind]
    for _ in range(args.warmup):
        fn()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        fn()
    dt = (time.perf_counter() - t0) / args.steps
    value = n / dt
    line = {"impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": cfgname},
            "cpu_baseline": {"value": value, "unit": unit, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="moin", choices=["moin", "reference"])
    ap.add_argument("--workload", default="decode", choices=["decode", "prefill", "router", "forward", "kmeans"])
    ap.add_argument("--no-graph", action="store_true", help="time plain launches instead of CUDA-graph replays")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-router-extra", action="store_true")
    ap.add_argument("--no-side-workloads", action="store_true", help="decode line without the prefill / forward keys")
    ap.add_argument("--print-timeline", action="store_true",
                    help="also print the kernel timeline of one step (start / end / duration in us) to stderr")
    ap.add_argument("--forward-layers", type=int, default=22)
    ap.add_argument("--no-group", action="store_true", help="one moin_lora_linear call per projection")
    ap.add_argument("--cache-slots", type=int, default=None,
                    help="decode / prefill through the two-tier adapter store with this many device slots (side "
                         "measurement: the step then contains a host round trip and the copies of the missing adapters)")
    ap.add_argument("--rank", type=int, default=None, help="decode / prefill at another LoRA rank than the config's (side measurement)")
    args = ap.parse_args()
    defaults = {"decode": (3000, 20), "prefill": (100, 5), "router": (50, 5), "forward": (5, 3), "kmeans": (50, 5)}
    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 5
        args.warmup = args.warmup if args.warmup is not None else 1
        return run_reference(args)
    if args.steps is None:
        args.steps = defaults[args.workload][0]
    if args.warmup is None:
        args.warmup = defaults[args.workload][1]

    import paper_2410_09687_b200 as moin
    if not os.path.exists(moin.lib_path()):
        from paper_2410_09687_b200 import build
        build.build()
    moin.lib()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    world, rank, local = dist_setup(args.gpus)
    dev = f"cuda:{local}"
    peaks = load_peaks()
    kind = args.workload
    if kind in ("decode", "prefill"):
        wl = LayerWorkload(kind, dev, grouped=not args.no_group, rank=args.rank, cache_slots=args.cache_slots)
    elif kind == "router":
        wl = RouterWorkload(dev)
    elif kind == "kmeans":
        wl = KMeansWorkload(dev)
    else:
        wl = ForwardWorkload(dev, n_layers=args.forward_layers)
    torch.cuda.synchronize()
    use_graph = (not args.no_graph) and kind != "forward" and not getattr(args, "cache_slots", None)

    sampler = ClockSampler(local)
    sampler.start()
    ms, graphed = timed_loop(world, wl.step, args.steps, args.warmup, use_graph)
    clocks = sampler.stop()
    ms = max_over_ranks(world, ms)
    value = whole_job_value(world, wl.units_per_step, ms)

    e2e_steps = max(5, args.steps // 4)
    e2e_mode = "one step after the other"
    if kind == "decode" and use_graph and wl.cache is None:
        # pipelined: blocks of E2E_BLOCK steps, the copies of a step beside the kernels of its neighbours
        blocks = max(2, e2e_steps // wl.E2E_BLOCK)
        ms_blk, _ = timed_loop(world, wl.e2e_block, blocks, 3, True)
        ms_e2e = ms_blk / wl.E2E_BLOCK
        e2e_mode = (f"copy-in / kernel / copy-out streams over {wl.E2E_LANES} buffer sets, one packed copy each way per step, "
                    f"CUDA graphs of {wl.E2E_BLOCK} steps")
    else:
        ms_e2e, _ = timed_loop(world, wl.step_e2e, e2e_steps, max(3, args.warmup // 2), use_graph)
    ms_e2e = max_over_ranks(world, ms_e2e)

    # per-kernel timing -> roofline of the dominant kernel
    agg, launches_per_step = profile_pass(moin, wl.step, min(args.steps, 20))
    # dominant kernel = most device time among the kernels on the call's own stream; in the short-segment
    # (decode) path the base GEMMs run on side streams beside the shrink, so their brackets overlap it
    on_path = {k: v for k, v in agg.items() if not (kind == "decode" and k in ("gemm_tc", "gemm_warp"))}
    top = max(on_path.items(), key=lambda kv: kv[1]["ms"])[0]
    kernels = {k: {"launches": a["launches"], "ms_per_launch": a["ms"] / max(a["launches"], 1)} for k, a in agg.items()}
    tl = kernel_timeline(wl.step, use_graph) if (rank == 0 and kind != "forward" and wl_cache_free(wl)) else None
    path = critical_path(*tl) if tl else None
    if tl and args.print_timeline:
        sys.stderr.write("kernel timeline of one step (us from the step's first kernel): start end duration name\n")
        for name, a, b in tl[0]:
            sys.stderr.write(f"{a:9.2f} {b:9.2f} {b - a:8.2f}  {name.split('(')[0][:90]}\n")
        sys.stderr.write(f"step span {tl[1]:.2f} us\n")
    prof_steps = min(args.steps, 20)
    roof = None
    extra = {}
    if kind in ("decode", "prefill") and wl.cache is not None and wl.cache_steps:
        extra["adapter_cache"] = {"slots": wl.cache.n_slots, "experts": wl.E,
                                  "misses_per_step": wl.cache_misses / wl.cache_steps,
                                  "h2d_adapter_bytes_per_step": wl.cache_bytes / wl.cache_steps}
    if kind in ("decode", "prefill"):
        nd = wl.distinct()
        alg = wl.algorithmic(nd)
        t_hbm = alg["step_bytes"] / (peaks["hbm_gbs"] * 1e9)
        t_tc = alg["step_flops"] / (peaks["bf16_tflops"] * 1e12)
        bound_time = max(t_hbm, t_tc)
        extra["step_roofline"] = {"bound": "hbm" if t_hbm >= t_tc else "tensor", "algorithmic_bytes": alg["step_bytes"],
                                  "algorithmic_flops": alg["step_flops"], "roofline_ms": bound_time * 1e3,
                                  "frac": bound_time * 1e3 / ms,
                                  "frac_nominal": max(alg["step_bytes"] / (NOMINAL_HBM_GBS * 1e9),
                                                      alg["step_flops"] / (NOMINAL_BF16_TFLOPS * 1e12)) * 1e3 / ms,
                                  "distinct_experts": nd}
        name_to_key = {"lora_expand_stream": "expand", "lora_shrink_stream": "shrink", "gemm_warp": "gemm", "gemm_tc": "gemm"}
        if top in name_to_key:
            a = agg[top]
            bytes_per_launch = alg["per_kernel_bytes"][name_to_key[top]] * prof_steps / a["launches"]
            sec = a["ms"] * 1e-3 / a["launches"]
            ach = bytes_per_launch / sec / 1e9
            roof = {"kernel": top, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": ach / peaks["hbm_gbs"], "frac_nominal": ach / NOMINAL_HBM_GBS, "peak_source": peaks["source"],
                    "algorithmic_bytes_per_launch": bytes_per_launch, "avg_launch_ms": sec * 1e3,
                    "traffic": traffic_for(top, kind)}
        elif top in ("lora_fused_tc", "lora_shrink_tc"):
            roof = tensor_roofline(top, agg[top], alg, prof_steps, peaks, kind)
    elif kind in ("router", "kmeans"):
        alg = wl.algorithmic()
        a = agg[top]
        sec = a["ms"] * 1e-3 / a["launches"]
        if kind == "kmeans" and "kmeans_update" in agg:
            u = agg["kmeans_update"]
            usec = u["ms"] * 1e-3 / u["launches"]
            extra["kmeans_update"] = {"bound": "hbm", "achieved": alg["update_bytes"] / usec / 1e9, "unit": "GB/s",
                                      "peak": peaks["hbm_gbs"], "frac": alg["update_bytes"] / usec / 1e9 / peaks["hbm_gbs"],
                                      "algorithmic_bytes_per_launch": alg["update_bytes"], "avg_launch_ms": usec * 1e3}
        ach = alg["flops"] / sec / 1e12
        tensor = top == "route_tc"
        roof = {"kernel": top, "bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": ach / peaks["bf16_tflops"], "frac_nominal": ach / NOMINAL_BF16_TFLOPS,
                "peak_source": peaks["source"] + " (burst)", "algorithmic_flops_per_launch": alg["flops"],
                "avg_launch_ms": sec * 1e3, "traffic": traffic_for(top, kind), "tensor_core_kernel": tensor}
    else:
        alg = wl.algorithmic()
        ach = alg["flops"] / (ms * 1e-3) / 1e12
        roof = {"kernel": "whole forward (" + top + " dominant)", "bound": "tensor", "achieved": ach,
                "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops_sustained"],
                "frac_nominal": ach / NOMINAL_BF16_TFLOPS, "peak_source": peaks["source"] + " (sustained)",
                "algorithmic_flops_per_launch": alg["flops"], "avg_launch_ms": ms, "traffic": None}
    if roof is None:
        a = agg[top]
        roof = {"kernel": top, "bound": "hbm", "achieved": None, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": None,
                "traffic": None, "avg_launch_ms": a["ms"] / a["launches"]}

    # secondary number of the metric: router queries/s on the router-stress configuration
    if kind == "decode" and rank == 0 and not args.no_router_extra:
        rw = RouterWorkload(dev)
        rms, _ = timed_loop(1, rw.step, 10, 3, False)
        ragg, _ = profile_pass(moin, rw.step, 3)
        rtop = max(ragg.items(), key=lambda kv: kv[1]["ms"])
        ralg = rw.algorithmic()
        rsec = rtop[1]["ms"] * 1e-3 / rtop[1]["launches"]
        extra["router_stress"] = {"queries_per_s": rw.Q / (rms * 1e-3), "ms_per_step": rms, "kernel": rtop[0],
                                  "achieved_tflops": ralg["flops"] / rsec / 1e12,
                                  "frac": ralg["flops"] / rsec / 1e12 / peaks["bf16_tflops"],
                                  "workload": rw.config()["workload"]}
        del rw
        torch.cuda.empty_cache()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and kind != "forward":
        import oracle
        oracle.build()
        if kind == "router":
            n, t = adaptive_oracle(wl.oracle_sample, 64, 4096)
            cpu = {"value": n / t, "unit": "queries/s", "cores": oracle.num_threads(), "kind": "oracle",
                   "sample": f"{n} of {wl.Q} queries against all {wl.K} centroids, {t:.1f} s"}
        elif kind == "kmeans":
            n, t = adaptive_oracle(wl.oracle_sample, 64, 4096)
            cpu = {"value": n / t, "unit": "points/s", "cores": oracle.num_threads(), "kind": "oracle",
                   "sample": f"assign + update of {n} of {wl.N} points against all {wl.K} centroids, {t:.1f} s"}
        else:
            n, t = adaptive_oracle(wl.oracle_sample, 16, 16 * wl.T if kind == "decode" else 4096)
            cpu = {"value": n / t, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
                   "sample": f"route + 7 projections of {n} tokens (batches of at most {wl.T}, step size {wl.T}), {t:.1f} s"}

    if rank == 0 and kind in ("router", "decode", "prefill"):
        # queries of the first batch whose two best cosines are closer than 1e-4 (reported by the library itself)
        rq = wl.queries[0]
        m = moin.route_top2(wl.router, rq)["margin"]
        extra["near_ties"] = {"margin_below": 1e-4, "count": int((m < 1e-4).sum().item()), "of": int(rq.shape[0]),
                              "min_margin": float(m.min().item())}
    if kind == "decode" and rank == 0 and world == 1 and not args.no_side_workloads and wl.cache is None and not args.rank:
        # the other headline workloads, so that one line carries all of them (their own runs: --workload ...)
        extra["prefill"] = side_prefill(moin, dev, peaks, local)
        extra["forward"] = side_forward(moin, dev, peaks, local)
    if rank == 0:
        metric = {"router": "router_queries_per_s", "kmeans": "kmeans_points_per_s"}.get(kind, "routed_lora_tokens_per_s")
        cfg = wl.config()
        cfg.update({"launch": "cuda_graph replay of one step" if graphed else "plain stream launches",
                    "replicas": world, "peaks": peaks})
        line = {"metric": metric, "value": value, "unit": wl.unit + "/s", "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": cfg, "clocks": clocks,
                "e2e": {"value": whole_job_value(world, wl.units_per_step, ms_e2e), "unit": wl.unit + "/s",
                        "h2d_bytes_per_step": wl.h2d, "d2h_bytes_per_step": wl.d2h, "ms_per_step": ms_e2e,
                        "pipelining": e2e_mode},
                "gpu_launches": int(round(launches_per_step * args.steps)), "roofline": roof, "kernels": kernels,
                "critical_path_us": path, "cpu_baseline": cpu}
        line.update(extra)
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
