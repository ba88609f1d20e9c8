"""ctypes binding of libmoin.so (include/moin.h).  Same names as the C entry points, torch
tensors in place of raw pointers.  Argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmoin.so")
_lib: Optional[ctypes.CDLL] = None

PLAN_AUTO, PLAN_SEGMENTS, PLAN_TILES = 0, 1, 2
LOGITS_ALL, LOGITS_LAST, LOGITS_NONE = 0, 1, 2
OPT_GEMM_IMPL = 1
OPT_NVTX = 3
ACT_NONE, ACT_RELU, ACT_SILU, ACT_GELU = 0, 1, 2, 3

EXPORTED_SYMBOLS = (
    "moin_status_string", "moin_version", "moin_last_cuda_error", "moin_device_status", "moin_device_status_reset",
    "moin_set_option", "moin_router_prepare", "moin_route_workspace_bytes", "moin_route", "moin_plan_bytes",
    "moin_plan_build", "moin_plan_read", "moin_lora_linear_workspace_bytes", "moin_lora_linear",
    "moin_decoder_workspace_bytes", "moin_decoder_forward", "moin_profile_enable", "moin_profile_read",
    "moin_kernel_name", "moin_route_static", "moin_lora_linear_group", "moin_lora_linear_group_workspace_bytes",
    "moin_kmeans_update", "moin_route_top2", "moin_route_top2_workspace_bytes", "moin_cache_create", "moin_cache_destroy", "moin_cache_admit", "moin_cache_slot_of",
    "moin_selftest_bounded_wait", "moin_decoder_forward_per_token", "moin_dequant_fp8", "moin_pool_set_adapter",
)


class MoinError(RuntimeError):
    pass


class _Router(ctypes.Structure):
    _fields_ = [("centroids", ctypes.c_void_p), ("inv_norm", ctypes.c_void_p), ("centroid_to_expert", ctypes.c_void_p),
                ("K", ctypes.c_int32), ("D", ctypes.c_int32)]


class _Pool(ctypes.Structure):
    _fields_ = [("A", ctypes.c_void_p), ("B", ctypes.c_void_p), ("slot_of_expert", ctypes.c_void_p),
                ("E", ctypes.c_int32), ("n_slots", ctypes.c_int32), ("r", ctypes.c_int32), ("d_in", ctypes.c_int32),
                ("d_out", ctypes.c_int32), ("activation", ctypes.c_int32), ("slot_rank", ctypes.c_void_p)]


class _Job(ctypes.Structure):
    _fields_ = [("x", ctypes.c_void_p), ("W", ctypes.c_void_p), ("pool", ctypes.POINTER(_Pool)), ("y", ctypes.c_void_p)]


class _CacheProj(ctypes.Structure):
    _fields_ = [("host_A", ctypes.c_void_p), ("host_B", ctypes.c_void_p), ("dev_A", ctypes.c_void_p),
                ("dev_B", ctypes.c_void_p), ("r", ctypes.c_int32), ("d_in", ctypes.c_int32), ("d_out", ctypes.c_int32)]


class _Plan(ctypes.Structure):
    _fields_ = [("buffer", ctypes.c_void_p), ("buffer_bytes", ctypes.c_size_t), ("T", ctypes.c_int32),
                ("E", ctypes.c_int32), ("mode", ctypes.c_int32), ("n_segments", ctypes.c_int32),
                ("n_tiles", ctypes.c_int32), ("n_lora_tokens", ctypes.c_int32), ("max_segment", ctypes.c_int32)]


class _Model(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("n_layers", "hidden", "n_heads", "n_kv_heads", "head_dim", "ffn", "vocab")] + \
               [(n, ctypes.c_float) for n in ("rms_eps", "rope_base", "lora_scale")] + \
               [("embed", ctypes.c_void_p), ("lm_head", ctypes.c_void_p), ("final_norm", ctypes.c_void_p),
                ("attn_norm", ctypes.POINTER(ctypes.c_void_p)), ("mlp_norm", ctypes.POINTER(ctypes.c_void_p)),
                ("W", ctypes.POINTER(ctypes.c_void_p)), ("pools", ctypes.POINTER(_Pool)), ("E", ctypes.c_int32),
                ("W8", ctypes.POINTER(ctypes.c_void_p)), ("W_scale", ctypes.POINTER(ctypes.c_void_p))]


class _Taps(ctypes.Structure):
    _fields_ = [("hidden_in", ctypes.c_void_p), ("hidden_out", ctypes.c_void_p), ("layer_begin", ctypes.c_int32),
                ("layer_end", ctypes.c_int32)]


class _ProfRec(ctypes.Structure):
    _fields_ = [("kernel", ctypes.c_int32), ("launches", ctypes.c_int32), ("ms", ctypes.c_float)]


class _DevStatus(ctypes.Structure):
    _fields_ = [("timeout_flag", ctypes.c_int32), ("timeout_site", ctypes.c_int32),
                ("invalid_expert_ids", ctypes.c_int32), ("reserved", ctypes.c_int32 * 5)]


def lib_path() -> str:
    return _LIB_PATH


def lib() -> ctypes.CDLL:
    """Loads libmoin.so (built in-tree by paper_2410_09687_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise MoinError(f"{_LIB_PATH} not found: build it with `python -m paper_2410_09687_b200.build` "
                            "(there is no fallback path)")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32, sz, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t, ctypes.c_float
        L.moin_status_string.restype = ctypes.c_char_p
        L.moin_status_string.argtypes = [i32]
        L.moin_version.restype = i32
        L.moin_last_cuda_error.restype = i32
        L.moin_device_status.argtypes = [ctypes.POINTER(_DevStatus), vp]
        L.moin_device_status_reset.argtypes = [vp]
        L.moin_set_option.argtypes = [i32, i32]
        L.moin_selftest_bounded_wait.argtypes = [i32, vp, vp]
        L.moin_router_prepare.argtypes = [vp, i32, i32, vp, vp]
        L.moin_route_workspace_bytes.restype = sz
        L.moin_route_workspace_bytes.argtypes = [i32, i32, i32]
        L.moin_route.argtypes = [ctypes.POINTER(_Router), vp, i32, vp, vp, vp, vp, sz, vp]
        L.moin_route_static.argtypes = [ctypes.POINTER(_Router), vp, i32, vp, vp, vp, vp]
        L.moin_kmeans_update.argtypes = [ctypes.POINTER(_Plan), vp, vp, vp, vp, i32, vp]
        L.moin_route_top2_workspace_bytes.restype = sz
        L.moin_route_top2_workspace_bytes.argtypes = [i32, i32, i32]
        L.moin_route_top2.argtypes = [ctypes.POINTER(_Router), vp, i32, vp, vp, vp, vp, vp, vp, sz, vp]
        L.moin_cache_create.argtypes = [i32, i32, ctypes.POINTER(_CacheProj), i32, vp, ctypes.POINTER(vp)]
        L.moin_cache_destroy.restype = None
        L.moin_cache_destroy.argtypes = [vp]
        L.moin_cache_admit.argtypes = [vp, vp, i32, vp, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_uint64)]
        L.moin_cache_slot_of.argtypes = [vp, i32, ctypes.POINTER(i32)]
        L.moin_plan_bytes.restype = sz
        L.moin_plan_bytes.argtypes = [i32, i32]
        L.moin_plan_build.argtypes = [vp, ctypes.POINTER(_Plan), vp]
        L.moin_plan_read.argtypes = [ctypes.POINTER(_Plan)] + [vp] * 9
        L.moin_lora_linear_workspace_bytes.restype = sz
        L.moin_lora_linear_workspace_bytes.argtypes = [i32, i32, i32, i32]
        L.moin_lora_linear.argtypes = [ctypes.POINTER(_Plan), vp, vp, ctypes.POINTER(_Pool), f32, i32, i32, i32, vp,
                                       vp, sz, vp]
        L.moin_lora_linear_group_workspace_bytes.restype = sz
        L.moin_lora_linear_group_workspace_bytes.argtypes = [i32, ctypes.POINTER(_Job), i32]
        L.moin_lora_linear_group.argtypes = [ctypes.POINTER(_Plan), ctypes.POINTER(_Job), i32, f32, vp, sz, vp]
        L.moin_decoder_workspace_bytes.restype = sz
        L.moin_decoder_workspace_bytes.argtypes = [ctypes.POINTER(_Model), i32, i32]
        L.moin_decoder_forward.argtypes = [ctypes.POINTER(_Model), vp, vp, vp, i32, i32, i32, vp, i32,
                                           ctypes.POINTER(_Taps), vp, sz, vp]
        L.moin_decoder_forward_per_token.argtypes = L.moin_decoder_forward.argtypes
        L.moin_dequant_fp8.argtypes = [vp, vp, i32, i32, vp, vp]
        L.moin_pool_set_adapter.argtypes = [ctypes.POINTER(_Pool), i32, i32, vp, vp, vp]
        L.moin_profile_enable.argtypes = [i32]
        L.moin_profile_read.argtypes = [ctypes.POINTER(_ProfRec), i32, ctypes.POINTER(i32)]
        L.moin_kernel_name.restype = ctypes.c_char_p
        L.moin_kernel_name.argtypes = [i32]
        for name in EXPORTED_SYMBOLS:
            fn = getattr(L, name)
            if fn.restype is ctypes.c_int:  # default restype: these return moin_status
                fn.restype = i32
        _lib = L
    return _lib


def _check(st: int, what: str) -> None:
    if st != 0:
        L = lib()
        raise MoinError(f"{what}: {L.moin_status_string(st).decode()} (cuda error {L.moin_last_cuda_error()})")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise MoinError("tensor arguments must live on a CUDA device (no CPU path exists)")
    if not t.is_contiguous():
        raise MoinError("tensor arguments must be contiguous")
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def set_option(key: int, value: int) -> None:
    _check(lib().moin_set_option(key, value), "moin_set_option")


def device_status(stream=None) -> dict:
    st = _DevStatus()
    _check(lib().moin_device_status(ctypes.byref(st), _stream(stream)), "moin_device_status")
    return {"timeout_flag": st.timeout_flag, "timeout_site": st.timeout_site,
            "invalid_expert_ids": st.invalid_expert_ids}


def device_status_reset(stream=None) -> None:
    _check(lib().moin_device_status_reset(_stream(stream)), "moin_device_status_reset")


def selftest_bounded_wait(limit_us: int, stream=None) -> dict:
    """moin_selftest_bounded_wait: runs the expiry path of the library's bounded device-side wait once."""
    res = torch.full((3,), -1, dtype=torch.int32, device="cuda")
    _check(lib().moin_selftest_bounded_wait(int(limit_us), _ptr(res), _stream(stream)), "moin_selftest_bounded_wait")
    torch.cuda.synchronize()
    r = res.cpu().tolist()
    return {"first_wait_returned_ok": r[0], "second_wait_returned_ok": r[1], "waited_us": r[2]}


def profile_enable(capacity: int) -> None:
    """moin_profile_enable: per-kernel CUDA-event brackets inside the library (0 = off)."""
    _check(lib().moin_profile_enable(capacity), "moin_profile_enable")


def profile_read(capacity: int = 65536) -> List[dict]:
    """moin_profile_read: [{'kernel': name, 'launches': n, 'ms': t}, ...] in launch order (synchronises)."""
    recs = (_ProfRec * capacity)()
    n = ctypes.c_int32(0)
    _check(lib().moin_profile_read(recs, capacity, ctypes.byref(n)), "moin_profile_read")
    L = lib()
    return [{"kernel": L.moin_kernel_name(recs[i].kernel).decode(), "launches": recs[i].launches, "ms": recs[i].ms}
            for i in range(min(n.value, capacity))]


class Router:
    """moin_router: centroid table [K, D] bf16 (+ optional centroid->expert map) with its inverse norms."""

    def __init__(self, centroids: torch.Tensor, centroid_to_expert: Optional[torch.Tensor] = None, stream=None):
        assert centroids.dtype == torch.bfloat16 and centroids.dim() == 2
        self.centroids = centroids
        self.map = centroid_to_expert
        self.K, self.D = centroids.shape
        self.inv_norm = torch.empty(self.K, dtype=torch.float32, device=centroids.device)
        _check(lib().moin_router_prepare(_ptr(centroids), self.K, self.D, _ptr(self.inv_norm), _stream(stream)),
               "moin_router_prepare")
        self.c = _Router(_ptr(centroids), _ptr(self.inv_norm), _ptr(centroid_to_expert), self.K, self.D)
        self._ws: Optional[torch.Tensor] = None

    def workspace(self, Q: int) -> torch.Tensor:
        n = lib().moin_route_workspace_bytes(Q, self.K, self.D)
        if self._ws is None or self._ws.numel() < n:
            self._ws = torch.empty(n, dtype=torch.uint8, device=self.centroids.device)
        return self._ws


def route(router: Router, queries: torch.Tensor, out_expert: Optional[torch.Tensor] = None,
          out_centroid: Optional[torch.Tensor] = None, out_best_sim: Optional[torch.Tensor] = None, stream=None):
    """moin_route.  Returns out_expert (int32 [Q])."""
    assert queries.dtype == torch.bfloat16 and queries.dim() == 2 and queries.shape[1] == router.D
    Q = queries.shape[0]
    if out_expert is None:
        out_expert = torch.empty(Q, dtype=torch.int32, device=queries.device)
    ws = router.workspace(Q)
    _check(lib().moin_route(ctypes.byref(router.c), _ptr(queries), Q, _ptr(out_expert), _ptr(out_centroid),
                            _ptr(out_best_sim), _ptr(ws), ws.numel(), _stream(stream)), "moin_route")
    return out_expert


def route_top2(router: Router, queries: torch.Tensor, stream=None) -> dict:
    """moin_route_top2: best centroid, runner-up and the margin between their cosines."""
    assert queries.dtype == torch.bfloat16 and queries.dim() == 2 and queries.shape[1] == router.D
    Q, dev = queries.shape[0], queries.device
    out = {"expert": torch.empty(Q, dtype=torch.int32, device=dev), "centroid": torch.empty(Q, dtype=torch.int32, device=dev),
           "second": torch.empty(Q, dtype=torch.int32, device=dev), "best": torch.empty(Q, dtype=torch.float32, device=dev),
           "margin": torch.empty(Q, dtype=torch.float32, device=dev)}
    n = lib().moin_route_top2_workspace_bytes(Q, router.K, router.D)
    ws = torch.empty(max(n, 256), dtype=torch.uint8, device=dev)
    _check(lib().moin_route_top2(ctypes.byref(router.c), _ptr(queries), Q, _ptr(out["expert"]), _ptr(out["centroid"]),
                                 _ptr(out["second"]), _ptr(out["best"]), _ptr(out["margin"]), _ptr(ws), ws.numel(),
                                 _stream(stream)), "moin_route_top2")
    return out


ROUTE_STATIC_MAX_Q = 65536


def route_static(router: Router, queries: torch.Tensor, out_expert: torch.Tensor,
                 out_centroid: Optional[torch.Tensor] = None, out_best_sim: Optional[torch.Tensor] = None,
                 stream=None) -> torch.Tensor:
    """moin_route_static: the router for callers that may not allocate device memory.

    Same result as ``route``; the scratch lives inside the library (at most ROUTE_STATIC_MAX_Q queries per
    call).  This wrapper allocates nothing either: the caller passes every output tensor.  Calls share
    the built-in scratch, so calls that overlap on the GPU race - keep them ordered on one stream."""
    assert queries.dtype == torch.bfloat16 and queries.dim() == 2 and queries.shape[1] == router.D
    _check(lib().moin_route_static(ctypes.byref(router.c), _ptr(queries), queries.shape[0], _ptr(out_expert),
                                   _ptr(out_centroid), _ptr(out_best_sim), _stream(stream)), "moin_route_static")
    return out_expert


class AdapterCache:
    """moin_cache: all experts' adapters in host memory, ``n_slots`` of them resident in the device pools.

    ``host`` is a list of (A [E, r, d_in], B [E, d_out, r]) CPU bf16 tensors (pinned for asynchronous copies), one
    pair per projection.  The device pools (``self.pools``) share one expert -> slot table."""

    def __init__(self, host: Sequence[tuple], n_slots: int, device):
        self.host = [(A, B) for A, B in host]
        E = self.host[0][0].shape[0]
        self.E, self.n_slots = E, n_slots
        self.table = torch.full((E,), -1, dtype=torch.int32, device=device)
        self.pools, descs = [], (_CacheProj * len(self.host))()
        for i, (A, B) in enumerate(self.host):
            assert A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16 and not A.is_cuda and not B.is_cuda
            assert A.is_contiguous() and B.is_contiguous() and A.shape[0] == E and B.shape[0] == E
            _, r, d_in = A.shape
            d_out = B.shape[1]
            dA = torch.zeros(n_slots, r, d_in, dtype=torch.bfloat16, device=device)
            dB = torch.zeros(n_slots, d_out, r, dtype=torch.bfloat16, device=device)
            self.pools.append(Pool(dA, dB, self.table))
            descs[i] = _CacheProj(A.data_ptr(), B.data_ptr(), dA.data_ptr(), dB.data_ptr(), r, d_in, d_out)
        h = ctypes.c_void_p()
        _check(lib().moin_cache_create(E, n_slots, descs, len(self.host), _ptr(self.table), ctypes.byref(h)),
               "moin_cache_create")
        self.handle = h

    def admit(self, expert_ids, stream=None) -> dict:
        """moin_cache_admit with the batch's expert ids (host int32 array-like).  Returns misses and bytes copied."""
        import numpy as _np
        ids = _np.ascontiguousarray(expert_ids, dtype=_np.int32)
        missed, nbytes = ctypes.c_int32(0), ctypes.c_uint64(0)
        _check(lib().moin_cache_admit(self.handle, ids.ctypes.data, ids.shape[0], _stream(stream), ctypes.byref(missed),
                                      ctypes.byref(nbytes)), "moin_cache_admit")
        return {"missed": missed.value, "bytes": nbytes.value}

    def slot_of(self, expert: int) -> int:
        s = ctypes.c_int32(0)
        _check(lib().moin_cache_slot_of(self.handle, expert, ctypes.byref(s)), "moin_cache_slot_of")
        return s.value

    def close(self):
        if self.handle is not None:
            lib().moin_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def kmeans_update(plan: "Plan", x: torch.Tensor, centroids_old: torch.Tensor,
                  centroids_new: Optional[torch.Tensor] = None, inv_norm_new: Optional[torch.Tensor] = None,
                  stream=None) -> torch.Tensor:
    """moin_kmeans_update: centroid k <- mean of the points the plan groups under cluster k."""
    assert x.dtype == torch.bfloat16 and centroids_old.dtype == torch.bfloat16 and x.dim() == 2
    assert centroids_old.shape == (plan.E, x.shape[1]) and plan.T == x.shape[0]
    if centroids_new is None:
        centroids_new = torch.empty_like(centroids_old)
    _check(lib().moin_kmeans_update(ctypes.byref(plan.c), _ptr(x), _ptr(centroids_old), _ptr(centroids_new),
                                    _ptr(inv_norm_new), x.shape[1], _stream(stream)), "moin_kmeans_update")
    return centroids_new


class Pool:
    """moin_pool: stacked adapters of one projection."""

    def __init__(self, A: torch.Tensor, B: torch.Tensor, slot_of_expert: torch.Tensor,
                 slot_rank: Optional[torch.Tensor] = None, activation: int = ACT_NONE):
        assert A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16 and slot_of_expert.dtype == torch.int32
        assert slot_rank is None or (slot_rank.dtype == torch.int32 and slot_rank.shape[0] == A.shape[0])
        self.A, self.B, self.slot_of_expert, self.slot_rank, self.activation = A, B, slot_of_expert, slot_rank, activation
        n_slots, r, d_in = A.shape
        d_out = B.shape[1]
        assert B.shape[0] == n_slots and B.shape[2] == r
        self.E, self.n_slots, self.r, self.d_in, self.d_out = slot_of_expert.shape[0], n_slots, r, d_in, d_out
        self.c = _Pool(_ptr(A), _ptr(B), _ptr(slot_of_expert), self.E, n_slots, r, d_in, d_out, int(activation),
                       _ptr(slot_rank))


def pool_set_adapter(pool: Pool, expert: int, slot: int, A: Optional[torch.Tensor] = None,
                     B: Optional[torch.Tensor] = None, stream=None) -> None:
    """moin_pool_set_adapter: write one adapter (A [r, d_in], B [d_out, r], device or pinned host) into ``slot`` and
    map ``expert`` to it; slot = -1 unmaps the expert."""
    for t in (A, B):
        assert t is None or (t.dtype == torch.bfloat16 and t.is_contiguous() and (t.is_cuda or t.is_pinned()))
    pa = None if A is None else A.data_ptr()
    pb = None if B is None else B.data_ptr()
    _check(lib().moin_pool_set_adapter(ctypes.byref(pool.c), int(expert), int(slot), pa, pb, _stream(stream)),
           "moin_pool_set_adapter")


class Plan:
    """moin_plan with its device buffer."""

    def __init__(self, T: int, E: int, device, mode: int = PLAN_AUTO):
        self.T, self.E = T, E
        n = lib().moin_plan_bytes(T, E)
        self.buffer = torch.empty(max(n, 256), dtype=torch.uint8, device=device)
        self.c = _Plan(_ptr(self.buffer), self.buffer.numel(), T, E, mode, 0, 0, 0, 0)

    @property
    def mode(self) -> int:
        return self.c.mode

    def read(self, stream=None) -> dict:
        """moin_plan_read: host copies of the plan arrays (synchronises)."""
        import numpy as np
        T = self.T
        ns, nt = ctypes.c_int32(0), ctypes.c_int32(0)
        arrs = {k: np.zeros(T + 1, np.int32) for k in ("perm", "seg_expert", "seg_start", "tile_row0", "tile_rows",
                                                       "tile_expert")}
        _check(lib().moin_plan_read(ctypes.byref(self.c), ctypes.addressof(ns), ctypes.addressof(nt),
                                    *[arrs[k].ctypes.data for k in ("perm", "seg_expert", "seg_start", "tile_row0",
                                                                    "tile_rows", "tile_expert")],
                                    _stream(stream)), "moin_plan_read")
        S, NT = ns.value, nt.value
        return {"S": S, "n_tiles": NT, "perm": arrs["perm"][:T], "seg_expert": arrs["seg_expert"][:S],
                "seg_start": arrs["seg_start"][:S + 1], "tile_row0": arrs["tile_row0"][:NT],
                "tile_rows": arrs["tile_rows"][:NT], "tile_expert": arrs["tile_expert"][:NT]}


def plan_build(token_expert: torch.Tensor, E: int, mode: int = PLAN_AUTO, plan: Optional[Plan] = None,
               stream=None) -> Plan:
    """moin_plan_build."""
    assert token_expert.dtype == torch.int32 and token_expert.dim() == 1
    T = token_expert.shape[0]
    if plan is None:
        plan = Plan(T, E, token_expert.device, mode)
    else:
        assert plan.T == T and plan.E == E
        plan.c.mode = mode
    _check(lib().moin_plan_build(_ptr(token_expert), ctypes.byref(plan.c), _stream(stream)), "moin_plan_build")
    return plan


_ws_cache: dict = {}


def _workspace(device, nbytes: int) -> torch.Tensor:
    key = str(device)
    ws = _ws_cache.get(key)
    if ws is None or ws.numel() < nbytes:
        ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
        _ws_cache[key] = ws
    return ws


def lora_linear(plan: Optional[Plan], x: torch.Tensor, W: torch.Tensor, pool: Optional[Pool], scale: float,
                y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """moin_lora_linear.  Returns y (bf16 [T, d_out])."""
    assert x.dtype == torch.bfloat16 and W.dtype == torch.bfloat16 and x.dim() == 2 and W.dim() == 2
    T, d_in = x.shape
    d_out = W.shape[0]
    assert W.shape[1] == d_in
    if pool is not None:
        assert pool.d_in == d_in and pool.d_out == d_out
    if y is None:
        y = torch.empty(T, d_out, dtype=torch.bfloat16, device=x.device)
    r = pool.r if pool is not None else 8
    n = lib().moin_lora_linear_workspace_bytes(T, d_in, d_out, r)
    ws = workspace if workspace is not None else _workspace(x.device, n)
    use = plan is not None and pool is not None
    _check(lib().moin_lora_linear(ctypes.byref(plan.c) if use else None, _ptr(x), _ptr(W),
                                  ctypes.byref(pool.c) if use else None, float(scale), T, d_in, d_out, _ptr(y),
                                  _ptr(ws), ws.numel(), _stream(stream)), "moin_lora_linear")
    return y


class JobGroup:
    """moin_lora_job array for moin_lora_linear_group: up to 4 independent projections sharing one plan.

    ``jobs``: sequence of (x, W, pool, y) with y preallocated (bf16 [T, d_out])."""

    def __init__(self, jobs: Sequence[tuple]):
        assert 1 <= len(jobs) <= 4
        self._keep = list(jobs)
        self.n = len(jobs)
        self.c = (_Job * self.n)()
        for i, (x, W, pool, y) in enumerate(jobs):
            assert x.dtype == torch.bfloat16 and W.dtype == torch.bfloat16 and y.dtype == torch.bfloat16
            assert x.shape[1] == pool.d_in and W.shape == (pool.d_out, pool.d_in) and y.shape == (x.shape[0], pool.d_out)
            self.c[i] = _Job(_ptr(x), _ptr(W), ctypes.pointer(pool.c), _ptr(y))
        self.T = jobs[0][0].shape[0]
        self.device = jobs[0][0].device
        self.workspace_bytes = lib().moin_lora_linear_group_workspace_bytes(self.T, self.c, self.n)


def lora_linear_group(plan: Plan, group: JobGroup, scale: float, workspace: Optional[torch.Tensor] = None,
                      stream=None) -> None:
    """moin_lora_linear_group: every job's y = x W^T + scale (x A_e^T) B_e^T, merged launches."""
    ws = workspace if workspace is not None else _workspace(group.device, group.workspace_bytes)
    _check(lib().moin_lora_linear_group(ctypes.byref(plan.c), group.c, group.n, float(scale), _ptr(ws), ws.numel(),
                                        _stream(stream)), "moin_lora_linear_group")


PROJ_ORDER = ("q", "k", "v", "o", "gate", "up", "down")


class DecoderModel:
    """moin_model built from per-layer tensors.  ``W[l][name]``, ``pools[l][name]`` (Pool) or pools=None."""

    def __init__(self, cfg, embed, lm_head, final_norm, attn_norm: Sequence[torch.Tensor],
                 mlp_norm: Sequence[torch.Tensor], W: Sequence[dict], pools: Optional[Sequence[dict]], E: int,
                 lora_scale: float, W8: Optional[Sequence[dict]] = None, W_scale: Optional[Sequence[dict]] = None):
        """``W8[l][name]`` (uint8 codes) with ``W_scale[l][name]`` (fp32 per output row): quantised base; the entries
        of ``W`` for those projections may then be None."""
        nl = cfg.n_layers
        self._keep = [embed, lm_head, final_norm, list(attn_norm), list(mlp_norm), list(W), pools, W8, W_scale]
        self.cfg = cfg
        self._an = (ctypes.c_void_p * nl)(*[_ptr(t) for t in attn_norm])
        self._mn = (ctypes.c_void_p * nl)(*[_ptr(t) for t in mlp_norm])
        self._W = (ctypes.c_void_p * (nl * 7))(*[_ptr(W[l].get(p)) for l in range(nl) for p in PROJ_ORDER])
        self._pools = None
        if pools is not None:
            self._pools = (_Pool * (nl * 7))(*[pools[l][p].c for l in range(nl) for p in PROJ_ORDER])
        m = _Model()
        m.n_layers, m.hidden, m.n_heads, m.n_kv_heads = nl, cfg.hidden, cfg.n_heads, cfg.n_kv_heads
        m.head_dim, m.ffn, m.vocab = cfg.head_dim, cfg.ffn, cfg.vocab
        m.rms_eps, m.rope_base, m.lora_scale = cfg.rms_eps, cfg.rope_base, lora_scale
        m.embed, m.lm_head, m.final_norm = _ptr(embed), _ptr(lm_head), _ptr(final_norm)
        m.attn_norm = ctypes.cast(self._an, ctypes.POINTER(ctypes.c_void_p))
        m.mlp_norm = ctypes.cast(self._mn, ctypes.POINTER(ctypes.c_void_p))
        m.W = ctypes.cast(self._W, ctypes.POINTER(ctypes.c_void_p))
        if self._pools is not None:
            m.pools = ctypes.cast(self._pools, ctypes.POINTER(_Pool))
        m.E = E
        if W8 is not None:
            self._W8 = (ctypes.c_void_p * (nl * 7))(*[_ptr(W8[l].get(p)) for l in range(nl) for p in PROJ_ORDER])
            self._Ws = (ctypes.c_void_p * (nl * 7))(*[_ptr(W_scale[l].get(p)) for l in range(nl) for p in PROJ_ORDER])
            m.W8 = ctypes.cast(self._W8, ctypes.POINTER(ctypes.c_void_p))
            m.W_scale = ctypes.cast(self._Ws, ctypes.POINTER(ctypes.c_void_p))
        self.c = m
        self.device = embed.device
        self._ws: Optional[torch.Tensor] = None

    def workspace(self, R: int, T: int) -> torch.Tensor:
        n = lib().moin_decoder_workspace_bytes(ctypes.byref(self.c), R, T)
        if self._ws is None or self._ws.numel() < n:
            self._ws = torch.empty(n, dtype=torch.uint8, device=self.device)
        return self._ws


def dequant_fp8(codes: torch.Tensor, scale: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """moin_dequant_fp8: uint8 codes [d_out, d_in] and fp32 scale [d_out] -> bf16 weight [d_out, d_in]."""
    assert codes.dtype == torch.uint8 and scale.dtype == torch.float32 and codes.dim() == 2
    d_out, d_in = codes.shape
    if out is None:
        out = torch.empty(d_out, d_in, dtype=torch.bfloat16, device=codes.device)
    _check(lib().moin_dequant_fp8(_ptr(codes), _ptr(scale), d_out, d_in, _ptr(out), _stream(stream)), "moin_dequant_fp8")
    return out


def decoder_forward(model: DecoderModel, tokens: torch.Tensor, cu_seqlens: torch.Tensor,
                    req_expert: Optional[torch.Tensor], max_seqlen: int, logits_mode: int = LOGITS_ALL,
                    logits: Optional[torch.Tensor] = None, hidden_in: Optional[torch.Tensor] = None,
                    hidden_out: Optional[torch.Tensor] = None, layer_begin: int = 0, layer_end: Optional[int] = None,
                    stream=None, token_expert: Optional[torch.Tensor] = None) -> Optional[torch.Tensor]:
    """moin_decoder_forward, or moin_decoder_forward_per_token when ``token_expert`` ([T] int32) is given.
    Returns logits (bf16) or None for LOGITS_NONE."""
    R, T = cu_seqlens.shape[0] - 1, tokens.shape[0]
    cfg = model.cfg
    if logits is None and logits_mode != LOGITS_NONE:
        rows = T if logits_mode == LOGITS_ALL else R
        logits = torch.empty(rows, cfg.vocab, dtype=torch.bfloat16, device=tokens.device)
    taps = _Taps(_ptr(hidden_in), _ptr(hidden_out), layer_begin, cfg.n_layers if layer_end is None else layer_end)
    ws = model.workspace(R, T)
    if token_expert is not None:
        _check(lib().moin_decoder_forward_per_token(ctypes.byref(model.c), _ptr(tokens), _ptr(cu_seqlens),
                                                    _ptr(token_expert), R, T, max_seqlen, _ptr(logits), logits_mode,
                                                    ctypes.byref(taps), _ptr(ws), ws.numel(), _stream(stream)),
               "moin_decoder_forward_per_token")
        return logits
    _check(lib().moin_decoder_forward(ctypes.byref(model.c), _ptr(tokens), _ptr(cu_seqlens), _ptr(req_expert), R, T,
                                      max_seqlen, _ptr(logits), logits_mode, ctypes.byref(taps), _ptr(ws), ws.numel(),
                                      _stream(stream)), "moin_decoder_forward")
    return logits
