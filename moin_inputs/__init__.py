"""Seeded synthetic inputs for the MoIN serving hot path.

This module only *draws* inputs (Gaussian weights and activations, planted-cluster
query embeddings, expert-id distributions, request lengths).  It holds none of the
method's arithmetic: no similarity, no LoRA product, no bucketing.  Both the CPU
oracle's tests and the CUDA path's tests/benchmarks take their inputs from here so
that the two sides always see the same bytes.

All floating-point tensors are returned as ``torch.bfloat16`` (the storage type of
the path); ``bf16_bits`` gives the raw 16-bit patterns as a numpy ``uint16`` array
for consumers that do not speak torch dtypes.

Shapes follow the five workload families used throughout the repository:

* ``tiny_layer`` / ``tiny_router``  - one 256x256 layer, 8 rank-8 experts, 16 ragged requests;
  8 centroids and 16 queries of dimension 64.
* ``decode_batch``                  - seven TinyLlama-shaped projections, 500 rank-64 experts,
  256 single-token requests.
* ``prefill_batch``                 - the same projections, 5 000 rank-16 experts, 32 x 512 tokens,
  Zipf(1.1) request->expert draw.
* ``planted_router``                - planted-cluster router workload (K Gaussian means, queries
  = mean + noise, both L2-normalised).
* ``decoder_model`` / ``decoder_batch`` - random-init Llama-architecture decoder with an adapter
  pool on the seven projections of every block.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

# (name, d_in, d_out) of the seven per-block projections of a TinyLlama-1.1B-shaped decoder.
TINYLLAMA_PROJECTIONS: Tuple[Tuple[str, int, int], ...] = (
    ("q", 2048, 2048),
    ("k", 2048, 256),
    ("v", 2048, 256),
    ("o", 2048, 2048),
    ("gate", 2048, 5632),
    ("up", 2048, 5632),
    ("down", 5632, 2048),
)


def _mix(seed: int, *stream: int) -> int:
    """Fold a seed and a stream label into one 63-bit integer (splitmix-style)."""
    z = (seed & 0xFFFFFFFFFFFFFFFF) ^ 0x9E3779B97F4A7C15
    for s in stream:
        z = (z + 0x9E3779B97F4A7C15 + (s & 0xFFFFFFFFFFFFFFFF)) & 0xFFFFFFFFFFFFFFFF
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
        z = z ^ (z >> 31)
    return z & 0x7FFFFFFFFFFFFFFF


def np_rng(seed: int, *stream: int) -> np.random.Generator:
    return np.random.default_rng(_mix(seed, *stream))


def normal_bf16(shape: Sequence[int], std: float, seed: int, *stream: int,
                device: str | torch.device = "cpu", mean: float = 0.0,
                chunk_elems: int = 1 << 27) -> torch.Tensor:
    """N(mean, std^2) samples rounded to bf16, drawn on ``device`` from a seeded torch generator.

    Large tensors are drawn in chunks so the fp32 temporary stays small.  The stream of
    values depends on the device type (CPU and CUDA generators differ); within one run
    every consumer sees the same tensor.
    """
    device = torch.device(device)
    n = int(np.prod(shape)) if len(shape) else 1
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    gen = torch.Generator(device=device)
    gen.manual_seed(_mix(seed, *stream))
    for lo in range(0, n, chunk_elems):
        hi = min(n, lo + chunk_elems)
        t = torch.randn(hi - lo, generator=gen, device=device, dtype=torch.float32)
        if std != 1.0:
            t.mul_(std)
        if mean != 0.0:
            t.add_(mean)
        out[lo:hi] = t.to(torch.bfloat16)
    return out.view(*shape)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """Raw bit patterns of a bf16 tensor as a C-contiguous numpy uint16 array (host copy)."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a bf16 tensor to a numpy float64 array (host copy)."""
    return t.detach().cpu().to(torch.float64).numpy()


# --------------------------------------------------------------------------------------
# Router workloads
# --------------------------------------------------------------------------------------

@dataclasses.dataclass
class RouterCase:
    centroids: torch.Tensor            # [K, D] bf16
    queries: torch.Tensor              # [Q, D] bf16
    labels: Optional[torch.Tensor]     # [Q] int32 planted label, or None
    K: int
    D: int
    Q: int


def _l2_normalise_rows(t: torch.Tensor) -> torch.Tensor:
    return t / t.norm(dim=1, keepdim=True).clamp_min(1e-30)


def gaussian_router(K: int, Q: int, D: int, seed: int,
                    device: str | torch.device = "cpu") -> RouterCase:
    """Independent Gaussian centroids and queries, L2-normalised, then rounded to bf16."""
    device = torch.device(device)
    g = torch.Generator(device=device)
    g.manual_seed(_mix(seed, 101))
    c = _l2_normalise_rows(torch.randn(K, D, generator=g, device=device, dtype=torch.float32))
    q = _l2_normalise_rows(torch.randn(Q, D, generator=g, device=device, dtype=torch.float32))
    return RouterCase(c.to(torch.bfloat16), q.to(torch.bfloat16), None, K, D, Q)


def planted_router(K: int, Q: int, D: int, seed: int, noise: float = 0.3,
                   device: str | torch.device = "cpu", unit_centroid_noise: bool = False,
                   chunk: int = 8192) -> RouterCase:
    """Planted-cluster router workload.

    K cluster means mu_k ~ N(0, I_D); centroid c_k = mu_k/|mu_k|.  Each query draws a label
    uniformly, q = mu_label + noise * N(0, I_D), then is L2-normalised.  With
    ``unit_centroid_noise`` the noise is added to the *unit* centroid instead (a much harder,
    near-tie-rich variant used only as a parity stress).  Everything is rounded to bf16.
    """
    device = torch.device(device)
    g = torch.Generator(device=device)
    g.manual_seed(_mix(seed, 202))
    mu = torch.randn(K, D, generator=g, device=device, dtype=torch.float32)
    c = _l2_normalise_rows(mu)
    labels = torch.randint(0, K, (Q,), generator=g, device=device, dtype=torch.int64)
    q = torch.empty(Q, D, dtype=torch.bfloat16, device=device)
    src = c if unit_centroid_noise else mu
    for lo in range(0, Q, chunk):
        hi = min(Q, lo + chunk)
        z = torch.randn(hi - lo, D, generator=g, device=device, dtype=torch.float32)
        q[lo:hi] = _l2_normalise_rows(src[labels[lo:hi]] + noise * z).to(torch.bfloat16)
    return RouterCase(c.to(torch.bfloat16), q, labels.to(torch.int32), K, D, Q)


# --------------------------------------------------------------------------------------
# Routed LoRA layer workloads
# --------------------------------------------------------------------------------------

@dataclasses.dataclass
class AdapterPool:
    """Stacked adapters of ONE projection: A[n_slots, r, d_in], B[n_slots, d_out, r] (bf16) and
    the expert->slot table (int32, -1 = expert has no adapter)."""
    A: torch.Tensor
    B: torch.Tensor
    slot_of_expert: torch.Tensor
    E: int
    r: int
    d_in: int
    d_out: int

    @property
    def n_slots(self) -> int:
        return int(self.A.shape[0])


@dataclasses.dataclass
class LayerCase:
    name: str
    x: torch.Tensor                # [T, d_in] bf16
    W: torch.Tensor                # [d_out, d_in] bf16
    pool: AdapterPool
    token_expert: torch.Tensor     # [T] int32 (-1 = base only)
    scale: float
    T: int


def make_pool(E: int, r: int, d_in: int, d_out: int, seed: int, *stream: int,
              std_a: float = 0.02, std_b: float = 0.02, missing: Sequence[int] = (),
              device: str | torch.device = "cpu") -> AdapterPool:
    """Adapters for E experts; experts listed in ``missing`` get no slot (slot -1)."""
    missing = set(int(m) for m in missing)
    slot = np.full(E, -1, dtype=np.int32)
    kept = [e for e in range(E) if e not in missing]
    slot[kept] = np.arange(len(kept), dtype=np.int32)
    n_slots = max(1, len(kept))
    A = normal_bf16((n_slots, r, d_in), std_a, seed, *stream, 1, device=device)
    B = normal_bf16((n_slots, d_out, r), std_b, seed, *stream, 2, device=device)
    return AdapterPool(A, B, torch.from_numpy(slot).to(device), E, r, d_in, d_out)


def expand_request_experts(req_expert: np.ndarray, lengths: np.ndarray) -> np.ndarray:
    """Per-request expert ids -> per-token ids for packed (request-major) tokens."""
    return np.repeat(req_expert.astype(np.int32), lengths.astype(np.int64))


def zipf_experts(R: int, E: int, s: float, seed: int, *stream: int) -> np.ndarray:
    """R draws from Zipf(s) over ranks 1..E; rank -> expert id through a fixed random permutation."""
    rng = np_rng(seed, *stream, 7)
    p = 1.0 / np.power(np.arange(1, E + 1, dtype=np.float64), s)
    p /= p.sum()
    ranks = rng.choice(E, size=R, p=p)
    perm = np_rng(seed, *stream, 8).permutation(E)
    return perm[ranks].astype(np.int32)


def layer_case(name: str, T: int, d_in: int, d_out: int, pool: AdapterPool,
               token_expert: np.ndarray, scale: float, seed: int, *stream: int,
               device: str | torch.device = "cpu", std_w: float = 0.02) -> LayerCase:
    x = normal_bf16((T, d_in), 1.0, seed, *stream, 11, device=device)
    W = normal_bf16((d_out, d_in), std_w, seed, *stream, 12, device=device)
    te = torch.from_numpy(np.ascontiguousarray(token_expert, dtype=np.int32)).to(device)
    return LayerCase(name, x, W, pool, te, float(scale), int(T))


def tiny_layer(seed: int = 0, device: str | torch.device = "cpu") -> LayerCase:
    """One 256x256 layer, 8 rank-8 experts, scale 2.0, 16 requests of U{1..32} tokens."""
    rng = np_rng(seed, 1)
    lengths = rng.integers(1, 33, size=16)
    req_expert = rng.integers(0, 8, size=16).astype(np.int32)
    te = expand_request_experts(req_expert, lengths)
    pool = make_pool(8, 8, 256, 256, seed, 2, device=device)
    case = layer_case("tiny", int(lengths.sum()), 256, 256, pool, te, 2.0, seed, 3, device=device)
    case.lengths = lengths          # type: ignore[attr-defined]
    case.req_expert = req_expert    # type: ignore[attr-defined]
    return case


def tiny_router(seed: int = 0, device: str | torch.device = "cpu") -> RouterCase:
    return gaussian_router(8, 16, 64, seed, device=device)


def decode_batch(seed: int = 1, E: int = 500, r: int = 64, T: int = 256, scale: float = 2.0,
                 token_expert: Optional[np.ndarray] = None,
                 projections: Sequence[Tuple[str, int, int]] = TINYLLAMA_PROJECTIONS,
                 device: str | torch.device = "cpu") -> List[LayerCase]:
    """Single-token requests over the seven projections; ids uniform over E unless given."""
    if token_expert is None:
        token_expert = np_rng(seed, 20).integers(0, E, size=T).astype(np.int32)
    cases = []
    for p, (name, d_in, d_out) in enumerate(projections):
        pool = make_pool(E, r, d_in, d_out, seed, 30 + p, device=device)
        cases.append(layer_case(name, T, d_in, d_out, pool, token_expert, scale, seed, 40 + p,
                                device=device))
    return cases


def prefill_batch(seed: int = 2, E: int = 5000, r: int = 16, R: int = 32, L: int = 512,
                  scale: float = 2.0, zipf_s: float = 1.1,
                  projections: Sequence[Tuple[str, int, int]] = TINYLLAMA_PROJECTIONS,
                  device: str | torch.device = "cpu") -> List[LayerCase]:
    """R requests of L tokens, request expert ~ Zipf(zipf_s) over E (skewed segments)."""
    req_expert = zipf_experts(R, E, zipf_s, seed, 21)
    te = expand_request_experts(req_expert, np.full(R, L))
    cases = []
    for p, (name, d_in, d_out) in enumerate(projections):
        pool = make_pool(E, r, d_in, d_out, seed, 30 + p, device=device)
        c = layer_case(name, R * L, d_in, d_out, pool, te, scale, seed, 40 + p, device=device)
        c.req_expert = req_expert   # type: ignore[attr-defined]
        cases.append(c)
    return cases


# --------------------------------------------------------------------------------------
# Decoder workloads
# --------------------------------------------------------------------------------------

@dataclasses.dataclass
class DecoderConfig:
    n_layers: int = 22
    hidden: int = 2048
    n_heads: int = 32
    n_kv_heads: int = 4
    head_dim: int = 64
    ffn: int = 5632
    vocab: int = 32000
    rms_eps: float = 1e-5
    rope_base: float = 10000.0
    E: int = 500
    r: int = 64
    scale: float = 2.0

    def projections(self) -> Tuple[Tuple[str, int, int], ...]:
        h, kv = self.hidden, self.n_kv_heads * self.head_dim
        return (("q", h, self.n_heads * self.head_dim), ("k", h, kv), ("v", h, kv),
                ("o", self.n_heads * self.head_dim, h),
                ("gate", h, self.ffn), ("up", h, self.ffn), ("down", self.ffn, h))


@dataclasses.dataclass
class DecoderModel:
    cfg: DecoderConfig
    embed: torch.Tensor                       # [vocab, hidden] bf16
    lm_head: torch.Tensor                     # [vocab, hidden] bf16
    final_norm: torch.Tensor                  # [hidden] bf16
    attn_norm: List[torch.Tensor]             # per layer [hidden] bf16
    mlp_norm: List[torch.Tensor]              # per layer [hidden] bf16
    W: List[Dict[str, torch.Tensor]]          # per layer, per projection [d_out, d_in] bf16
    pools: List[Dict[str, AdapterPool]]       # per layer, per projection


def decoder_model(cfg: DecoderConfig, seed: int = 4, missing: Sequence[int] = (),
                  device: str | torch.device = "cpu") -> DecoderModel:
    """Random-init decoder: weights N(0, 0.02^2), norm gains 1 + N(0, 0.02^2), all bf16."""
    embed = normal_bf16((cfg.vocab, cfg.hidden), 0.02, seed, 1, device=device)
    lm_head = normal_bf16((cfg.vocab, cfg.hidden), 0.02, seed, 2, device=device)
    final_norm = normal_bf16((cfg.hidden,), 0.02, seed, 3, device=device, mean=1.0)
    attn_norm, mlp_norm, Ws, pools = [], [], [], []
    for l in range(cfg.n_layers):
        attn_norm.append(normal_bf16((cfg.hidden,), 0.02, seed, 10, l, device=device, mean=1.0))
        mlp_norm.append(normal_bf16((cfg.hidden,), 0.02, seed, 11, l, device=device, mean=1.0))
        Wl, Pl = {}, {}
        for p, (name, d_in, d_out) in enumerate(cfg.projections()):
            Wl[name] = normal_bf16((d_out, d_in), 0.02, seed, 12, l, p, device=device)
            Pl[name] = make_pool(cfg.E, cfg.r, d_in, d_out, seed, 13, l, p, missing=missing,
                                 device=device)
        Ws.append(Wl)
        pools.append(Pl)
    return DecoderModel(cfg, embed, lm_head, final_norm, attn_norm, mlp_norm, Ws, pools)


@dataclasses.dataclass
class DecoderBatch:
    tokens: torch.Tensor        # [T] int32
    cu_seqlens: torch.Tensor    # [R+1] int32
    req_expert: torch.Tensor    # [R] int32 (-1 = base only)
    R: int
    T: int


def decoder_batch(cfg: DecoderConfig, lengths: Sequence[int], seed: int = 4,
                  req_expert: Optional[Sequence[int]] = None,
                  device: str | torch.device = "cpu") -> DecoderBatch:
    lengths = np.asarray(lengths, dtype=np.int64)
    R, T = len(lengths), int(lengths.sum())
    rng = np_rng(seed, 50)
    tokens = rng.integers(0, cfg.vocab, size=T).astype(np.int32)
    if req_expert is None:
        req_expert = rng.integers(0, cfg.E, size=R)
    cu = np.zeros(R + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lengths)
    return DecoderBatch(torch.from_numpy(tokens).to(device), torch.from_numpy(cu).to(device),
                        torch.from_numpy(np.asarray(req_expert, dtype=np.int32)).to(device), R, T)


def distinct_experts(token_expert: np.ndarray) -> int:
    te = np.asarray(token_expert)
    return int(np.unique(te[te >= 0]).size)


__all__ = [n for n in dir() if not n.startswith("_")]
