"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not a product path).

Only ``tests/``, ``__graft_entry__.smoke()`` and the benchmark's CPU-baseline leg may import
this package.  It compiles ``moin_oracle.c`` with gcc on first use (``build()``) and
exposes thin numpy wrappers; every argument is a host numpy array.  Floating-point inputs
are either float64 arrays or bf16 bit patterns (``uint16`` arrays); outputs are float64 /
int32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moin_oracle.c")
_LIB = os.path.join(_HERE, "libmoin_oracle.so")
_lib: Optional[ctypes.CDLL] = None

F64, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle (plain C, -O2, OpenMP over independent units)."""
    if force or (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp,
                               _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Model(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_layers", "hidden", "n_heads", "n_kv_heads", "head_dim", "ffn", "vocab", "E", "r",
                 "n_slots")] + \
               [("rms_eps", ctypes.c_double), ("rope_base", ctypes.c_double), ("scale", ctypes.c_double),
                ("embed", ctypes.c_void_p), ("lm_head", ctypes.c_void_p), ("final_norm", ctypes.c_void_p),
                ("attn_norm", ctypes.POINTER(ctypes.c_void_p)), ("mlp_norm", ctypes.POINTER(ctypes.c_void_p)),
                ("W", ctypes.POINTER(ctypes.c_void_p)), ("A", ctypes.POINTER(ctypes.c_void_p)),
                ("B", ctypes.POINTER(ctypes.c_void_p)), ("slot_of_expert", ctypes.c_void_p)]


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        L.moin_oracle_num_threads.restype = ctypes.c_int
        L.moin_oracle_round_bf16.restype = ctypes.c_double
        L.moin_oracle_round_bf16.argtypes = [ctypes.c_double]
        L.moin_oracle_route.restype = ctypes.c_int
        L.moin_oracle_route.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int64,
                                        ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.moin_oracle_lora_linear.restype = ctypes.c_int
        L.moin_oracle_lora_linear.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int, ctypes.c_void_p,
                                                                     ctypes.c_void_p, ctypes.c_int64,
                                                                     ctypes.c_int64, ctypes.c_int,
                                                                     ctypes.c_int64, ctypes.c_int64,
                                                                     ctypes.c_double, ctypes.c_void_p]
        L.moin_oracle_lora_linear_ex.restype = ctypes.c_int
        L.moin_oracle_lora_linear_ex.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                                                        ctypes.c_void_p, ctypes.c_int, ctypes.c_int64,
                                                                        ctypes.c_int64, ctypes.c_int, ctypes.c_int64,
                                                                        ctypes.c_int64, ctypes.c_double, ctypes.c_void_p]
        L.moin_oracle_decoder_forward.restype = ctypes.c_int
        L.moin_oracle_decoder_forward.argtypes = [ctypes.POINTER(_Model), ctypes.c_void_p, ctypes.c_void_p,
                                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64,
                                                  ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.moin_oracle_e4m3_value.restype = ctypes.c_double
        L.moin_oracle_e4m3_value.argtypes = [ctypes.c_int]
        L.moin_oracle_dequant_fp8.restype = ctypes.c_int
        L.moin_oracle_dequant_fp8.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p]
        L.moin_oracle_bucket.restype = ctypes.c_int64
        L.moin_oracle_bucket.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                         ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.moin_oracle_kmeans_update.restype = ctypes.c_int
        L.moin_oracle_kmeans_update.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p,
                                                ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p,
                                                ctypes.c_void_p]
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().moin_oracle_num_threads())


def round_bf16(v: float) -> float:
    return float(lib().moin_oracle_round_bf16(float(v)))


def _fp(a: np.ndarray):
    """(contiguous array, dtype code) for a float64 or bf16-bits array."""
    if a.dtype == np.uint16:
        return np.ascontiguousarray(a), BF16
    return np.ascontiguousarray(a, dtype=np.float64), F64


def _same_kind(*arrs):
    out, kinds = [], set()
    for a in arrs:
        if a is None:
            out.append(None)
            continue
        b, k = _fp(a)
        out.append(b)
        kinds.add(k)
    if len(kinds) > 1:  # mixed: widen the bf16 ones exactly
        out = [None if a is None else (_bits_to_f64(a) if a.dtype == np.uint16 else a) for a in out]
        return out, F64
    return out, (kinds.pop() if kinds else F64)


def _bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def route(q: np.ndarray, c: np.ndarray, centroid_to_expert: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Cosine-argmax router.  Returns centroid ids, expert ids, best similarity, top-2 margin."""
    (q, c), kind = _same_kind(q, c)
    Q, D = q.shape
    K, D2 = c.shape
    assert D == D2
    m = None if centroid_to_expert is None else np.ascontiguousarray(centroid_to_expert, dtype=np.int32)
    cid = np.zeros(Q, np.int32)
    eid = np.zeros(Q, np.int32)
    best = np.zeros(Q, np.float64)
    margin = np.zeros(Q, np.float64)
    rc = lib().moin_oracle_route(_ptr(q), _ptr(c), kind, Q, K, D, _ptr(m), _ptr(cid), _ptr(eid), _ptr(best),
                                 _ptr(margin))
    if rc:
        raise RuntimeError(f"moin_oracle_route failed: {rc}")
    return {"centroid": cid, "expert": eid, "best": best, "margin": margin}


ACT_NONE, ACT_RELU, ACT_SILU, ACT_GELU = 0, 1, 2, 3


def lora_linear(x: np.ndarray, W: np.ndarray, A: Optional[np.ndarray], B: Optional[np.ndarray],
                token_expert: Optional[np.ndarray], slot_of_expert: Optional[np.ndarray], scale: float,
                slot_rank: Optional[np.ndarray] = None, act: int = ACT_NONE) -> np.ndarray:
    """y[T, d_out] (float64) of the routed LoRA layer; A [n_slots, r, d_in], B [n_slots, d_out, r].
    ``slot_rank`` ([n_slots] int32): rank of each slot's adapter (<= r; rows of A / columns of B beyond it are
    not read); ``act``: function applied between the two low-rank matrices."""
    (x, W, A, B), kind = _same_kind(x, W, A, B)
    T, d_in = x.shape
    d_out = W.shape[0]
    assert W.shape[1] == d_in
    r = 0 if A is None else A.shape[1]
    if A is not None:
        assert A.shape[2] == d_in and B.shape[1] == d_out and B.shape[2] == r and A.shape[0] == B.shape[0]
    te = None if token_expert is None else np.ascontiguousarray(token_expert, dtype=np.int32)
    so = None if slot_of_expert is None else np.ascontiguousarray(slot_of_expert, dtype=np.int32)
    if so is not None and A is not None and so.size:
        assert int(so.max()) < A.shape[0]
    E = 0 if so is None else so.shape[0]
    y = np.zeros((T, d_out), np.float64)
    if slot_rank is None and act == ACT_NONE:
        rc = lib().moin_oracle_lora_linear(_ptr(x), _ptr(W), _ptr(A), _ptr(B), kind, _ptr(te), _ptr(so), T, E, r,
                                           d_in, d_out, float(scale), _ptr(y))
    else:
        sr = None if slot_rank is None else np.ascontiguousarray(slot_rank, dtype=np.int32)
        if sr is not None and A is not None:
            assert sr.shape[0] == A.shape[0]
        rc = lib().moin_oracle_lora_linear_ex(_ptr(x), _ptr(W), _ptr(A), _ptr(B), kind, _ptr(te), _ptr(so), _ptr(sr),
                                              int(act), T, E, r, d_in, d_out, float(scale), _ptr(y))
    if rc:
        raise RuntimeError(f"moin_oracle_lora_linear failed: {rc}")
    return y


def e4m3_value(code: int) -> float:
    return float(lib().moin_oracle_e4m3_value(int(code)))


def dequant_fp8(codes: np.ndarray, scale: np.ndarray) -> np.ndarray:
    """bf16 bit patterns [d_out, d_in] of the weight a quantised base layer uses: bf16(fp32(value(code) * scale[row]))."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scale = np.ascontiguousarray(scale, dtype=np.float32)
    d_out, d_in = codes.shape
    assert scale.shape == (d_out,)
    out = np.zeros((d_out, d_in), np.uint16)
    rc = lib().moin_oracle_dequant_fp8(_ptr(codes), _ptr(scale), d_out, d_in, _ptr(out))
    if rc:
        raise RuntimeError(f"moin_oracle_dequant_fp8 failed: {rc}")
    return out


def bucket(token_expert: np.ndarray, slot_of_expert: np.ndarray, n_slots: int) -> Dict[str, np.ndarray]:
    te = np.ascontiguousarray(token_expert, dtype=np.int32)
    so = np.ascontiguousarray(slot_of_expert, dtype=np.int32)
    T = te.shape[0]
    perm = np.zeros(max(T, 1), np.int32)
    seg_slot = np.zeros(max(n_slots, 1), np.int32)
    seg_start = np.zeros(n_slots + 1, np.int32)
    S = lib().moin_oracle_bucket(_ptr(te), _ptr(so), T, so.shape[0], n_slots, _ptr(perm), _ptr(seg_slot),
                                 _ptr(seg_start))
    if S < 0:
        raise RuntimeError("moin_oracle_bucket failed")
    return {"perm": perm[:T], "seg_slot": seg_slot[:S], "seg_start": seg_start[:S + 1], "S": int(S)}


def kmeans_update(x: np.ndarray, c_old: np.ndarray, assign: np.ndarray) -> Dict[str, np.ndarray]:
    """K-means update step: mean of every cluster's members (float64); empty clusters keep c_old's row."""
    (x, c_old), kind = _same_kind(x, c_old)
    N, D = x.shape
    K = c_old.shape[0]
    assert c_old.shape[1] == D
    a = np.ascontiguousarray(assign, dtype=np.int32)
    assert a.shape == (N,)
    c_new = np.zeros((K, D), np.float64)
    counts = np.zeros(K, np.int64)
    rc = lib().moin_oracle_kmeans_update(_ptr(x), _ptr(c_old), kind, _ptr(a), N, K, D, _ptr(c_new), _ptr(counts))
    if rc:
        raise RuntimeError(f"moin_oracle_kmeans_update failed: {rc}")
    return {"centroids": c_new, "counts": counts}


PROJ_ORDER = ("q", "k", "v", "o", "gate", "up", "down")


class DecoderOracle:
    """Holds host copies (bf16 bits) of a decoder's weights and runs the oracle forward.

    ``weights``: dict with 'embed', 'lm_head', 'final_norm' (uint16 arrays), 'attn_norm',
    'mlp_norm' (lists), 'W', 'A', 'B' (lists over layers of dicts over PROJ_ORDER; A/B may be
    None for a base-only model), 'slot_of_expert' (int32 [E]).
    """

    def __init__(self, cfg, weights: dict):
        self.cfg = cfg
        self._keep: List[np.ndarray] = []
        nl = cfg.n_layers

        def keep(a, dt=np.uint16):
            a = np.ascontiguousarray(a, dtype=dt)
            self._keep.append(a)
            return a

        def parr(items: Sequence[Optional[np.ndarray]]):
            arr = (ctypes.c_void_p * len(items))()
            for i, a in enumerate(items):
                arr[i] = None if a is None else keep(a).ctypes.data
            self._keep.append(arr)
            return arr

        m = _Model()
        m.n_layers, m.hidden, m.n_heads, m.n_kv_heads = nl, cfg.hidden, cfg.n_heads, cfg.n_kv_heads
        m.head_dim, m.ffn, m.vocab, m.E, m.r = cfg.head_dim, cfg.ffn, cfg.vocab, cfg.E, cfg.r
        m.rms_eps, m.rope_base, m.scale = cfg.rms_eps, cfg.rope_base, cfg.scale
        m.embed = keep(weights["embed"]).ctypes.data
        m.lm_head = keep(weights["lm_head"]).ctypes.data
        m.final_norm = keep(weights["final_norm"]).ctypes.data
        self._an = parr(weights["attn_norm"])
        self._mn = parr(weights["mlp_norm"])
        self._W = parr([weights["W"][l][p] for l in range(nl) for p in PROJ_ORDER])
        has_ad = weights.get("A") is not None
        if has_ad:
            self._A = parr([weights["A"][l][p] for l in range(nl) for p in PROJ_ORDER])
            self._B = parr([weights["B"][l][p] for l in range(nl) for p in PROJ_ORDER])
            m.n_slots = int(weights["A"][0]["q"].shape[0])
        m.attn_norm = ctypes.cast(self._an, ctypes.POINTER(ctypes.c_void_p))
        m.mlp_norm = ctypes.cast(self._mn, ctypes.POINTER(ctypes.c_void_p))
        m.W = ctypes.cast(self._W, ctypes.POINTER(ctypes.c_void_p))
        if has_ad:
            m.A = ctypes.cast(self._A, ctypes.POINTER(ctypes.c_void_p))
            m.B = ctypes.cast(self._B, ctypes.POINTER(ctypes.c_void_p))
        so = weights.get("slot_of_expert")
        m.slot_of_expert = None if so is None else keep(so, np.int32).ctypes.data
        self._m = m

    def forward(self, tokens, cu_seqlens, req_expert, layer_begin: int = 0, layer_end: Optional[int] = None,
                round_storage: bool = False, hidden_in: Optional[np.ndarray] = None,
                want_hidden: bool = False, want_logits: bool = True, token_expert=None):
        """``token_expert`` ([T] int32): one expert per token instead of one per request (the paper's
        future-work variant, Sec. 5); ``req_expert`` is then ignored."""
        cfg = self.cfg
        layer_end = cfg.n_layers if layer_end is None else layer_end
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
        re_ = None if req_expert is None else np.ascontiguousarray(req_expert, dtype=np.int32)
        R, T = cu.shape[0] - 1, int(cu[-1])
        hin = None if hidden_in is None else np.ascontiguousarray(hidden_in, dtype=np.float64)
        hout = np.zeros((T, cfg.hidden), np.float64) if want_hidden else None
        logits = np.zeros((T, cfg.vocab), np.float64) if want_logits else None
        te_ = None if token_expert is None else np.ascontiguousarray(token_expert, dtype=np.int32)
        rc = lib().moin_oracle_decoder_forward(ctypes.byref(self._m), _ptr(tokens), _ptr(cu), _ptr(re_), _ptr(te_), R, T,
                                               layer_begin, layer_end, int(round_storage), _ptr(hin),
                                               _ptr(hout), _ptr(logits))
        if rc:
            raise RuntimeError(f"moin_oracle_decoder_forward failed: {rc}")
        return {"hidden": hout, "logits": logits}
