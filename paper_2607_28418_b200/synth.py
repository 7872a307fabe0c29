"""Seeded synthetic inputs for the WIDE hot path (shapes of Llama-style layers).

This module only draws random numbers and lays them out; it contains none of the
method's arithmetic (no routing, no reordering, no FFN).  The oracle, the CUDA
binding, the tests and the benchmark all take the host buffers produced here, so
both sides of every parity check see the same bytes.

Conventions
-----------
* Every array is generated on the host with ``numpy.random.default_rng(seed)``.
* ``dtype == "bf16"``: values are rounded to bfloat16 (round-to-nearest-even) and
  returned as float32 arrays whose low 16 mantissa bits are zero; ``to_bf16_bits``
  gives the uint16 payload for upload.  ``dtype == "fp32"``: plain float32.
* Weight layouts follow the paper's Linear convention C = A B^T with B in [N, K]
  (Section 3.1, FFN pruning unit): ``w_gate, w_up`` are [d_ff, hidden],
  ``w_down`` is [hidden, d_ff], ``w_o`` is [hidden, heads*head_dim], ``w_router``
  is [n_groups, hidden].
* "N(0, s)" in a workload description means standard deviation ``s``.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np


# --------------------------------------------------------------------------- bf16
def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result is float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    lsb = (bits >> 16) & 1
    bits = (bits + 0x7FFF + lsb) & 0xFFFF0000
    return bits.astype(np.uint32).view(np.float32).reshape(a.shape)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 payload of values that are already exactly representable in bfloat16."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    if np.any(bits & 0xFFFF):
        raise ValueError("array is not bf16-representable; call round_to_bf16 first")
    return (bits >> 16).astype(np.uint16).reshape(a.shape)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """float32 values of a uint16 bfloat16 payload."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).reshape(b.shape)


# --------------------------------------------------------------------------- configs
@dataclass(frozen=True)
class WideConfig:
    """One workload: a (possibly attention-augmented) FFN layer with a token router."""

    name: str
    tokens: int            # T (flattened batch * sequence)
    hidden: int            # D
    d_ff: int              # D'
    group: int             # G  (FFN channel-group size)
    k: int                 # active FFN groups per token
    dtype: str = "bf16"    # "bf16" | "fp32"
    router: str = "random"  # "random" | "clustered" | "clustered_corr"
    tile_m: int = 128
    # attention half (only configs that exercise the O-projection)
    attn_dim: int = 0      # H * d
    attn_group: int = 0    # heads_per_group * d
    attn_k: int = 0
    kv_heads: int = 0      # KV heads of 128 (0: as many as query heads)

    @property
    def n_groups(self) -> int:
        return self.d_ff // self.group

    @property
    def attn_n_groups(self) -> int:
        return self.attn_dim // self.attn_group if self.attn_group else 0

    def with_(self, **kw) -> "WideConfig":
        return replace(self, **kw)


CONFIGS: Dict[str, WideConfig] = {
    # Tiny masked FFN, fp32, the oracle runs it in well under a second.
    "tiny": WideConfig("tiny", tokens=128, hidden=256, d_ff=1024, group=64, k=8, dtype="fp32"),
    # Llama-7B-shaped FFN prefill (the benchmark workload).
    "llama7b_prefill": WideConfig("llama7b_prefill", tokens=2048, hidden=4096, d_ff=11008,
                                  group=128, k=43),
    # Llama-3-8B-shaped FFN decode (batch is varied by the caller: 1/8/32/64).
    "llama8b_decode": WideConfig("llama8b_decode", tokens=32, hidden=4096, d_ff=14336,
                                 group=128, k=56),
    # Sparsity / group-size sweep base point on the 8B-shaped FFN.
    "llama8b_prefill": WideConfig("llama8b_prefill", tokens=4096, hidden=4096, d_ff=14336,
                                  group=128, k=56),
    # Llama-2-13B-shaped layer: head-group masked O-projection + FFN.
    "llama13b_layer": WideConfig("llama13b_layer", tokens=4096, hidden=5120, d_ff=13824,
                                 group=128, k=54, attn_dim=5120, attn_group=512, attn_k=5),
    # Llama-3-8B-shaped layer: grouped-query attention (32 query heads on 8 KV heads of 128; a routing
    # group = the 4 query heads of one KV head) + the 8B FFN.
    "llama8b_layer": WideConfig("llama8b_layer", tokens=4096, hidden=4096, d_ff=14336,
                                group=128, k=56, attn_dim=4096, attn_group=512, attn_k=4, kv_heads=8),
}


def sweep_point(tokens: int, group: int, active_fraction: float, router: str) -> WideConfig:
    """One point of the sparsity sweep on the 8B-shaped FFN (k = round(p * N_G))."""
    n_groups = 14336 // group
    k = int(round(active_fraction * n_groups))
    return WideConfig(f"sweep_T{tokens}_G{group}_p{int(active_fraction * 100)}_{router}",
                      tokens=tokens, hidden=4096, d_ff=14336, group=group, k=k, router=router)


# --------------------------------------------------------------------------- generators
def _cast(a: np.ndarray, dtype: str) -> np.ndarray:
    a = a.astype(np.float32)
    return round_to_bf16(a) if dtype == "bf16" else a


def make_activations(rng: np.random.Generator, tokens: int, hidden: int, dtype: str,
                     router: str = "random") -> np.ndarray:
    """x ~ N(0,1).  Clustered variants: every token is a copy of one of 4 prototypes.

    ``clustered``      : prototypes independent N(0, I)
    ``clustered_corr`` : prototypes sqrt(0.9)*s + sqrt(0.1)*e_c with a shared s, so the
                         four masks overlap strongly and the union of groups stays small.
    """
    if router == "random":
        x = rng.standard_normal((tokens, hidden), dtype=np.float32)
    else:
        protos = rng.standard_normal((4, hidden), dtype=np.float32)
        if router == "clustered_corr":
            shared = rng.standard_normal((1, hidden), dtype=np.float32)
            protos = np.sqrt(0.9, dtype=np.float32) * shared + np.sqrt(0.1, dtype=np.float32) * protos
        elif router != "clustered":
            raise ValueError(f"unknown router variant {router!r}")
        which = rng.integers(0, 4, size=tokens)
        x = protos[which]
    return _cast(x, dtype)


def make_weight(rng: np.random.Generator, rows: int, cols: int, std: float, dtype: str) -> np.ndarray:
    w = rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(std)
    return _cast(w, dtype)


def make_ffn_case(cfg: WideConfig, seed: int, tokens: Optional[int] = None) -> Dict[str, np.ndarray]:
    """Host buffers for route -> reorder -> masked FFN on ``cfg``.

    Keys: x [T, D], w_router [N_G, D], w_gate [D', D], w_up [D', D], w_down [D, D'].
    Router rows ~ N(0, 1/sqrt(D)) so scores have unit variance and the top-k masks are
    close to uniformly random; FFN weights ~ N(0, 0.02).
    """
    T = cfg.tokens if tokens is None else tokens
    rng = np.random.default_rng(seed)
    out = {
        "x": make_activations(rng, T, cfg.hidden, cfg.dtype, cfg.router),
        "w_router": make_weight(rng, cfg.n_groups, cfg.hidden, 1.0 / np.sqrt(cfg.hidden), cfg.dtype),
        "w_gate": make_weight(rng, cfg.d_ff, cfg.hidden, 0.02, cfg.dtype),
        "w_up": make_weight(rng, cfg.d_ff, cfg.hidden, 0.02, cfg.dtype),
        "w_down": make_weight(rng, cfg.hidden, cfg.d_ff, 0.02, cfg.dtype),
    }
    return out


def make_oproj_case(cfg: WideConfig, seed: int, tokens: Optional[int] = None) -> Dict[str, np.ndarray]:
    """Host buffers for route -> reorder -> head-group-masked O-projection.

    Keys: x [T, D] (router input: the layer's hidden state), attn_out [T, H*d] ~ N(0,1)
    drawn independently of x, w_router_attn [N_G, D], w_o [D, H*d].
    """
    if not cfg.attn_group:
        raise ValueError(f"config {cfg.name} has no attention half")
    T = cfg.tokens if tokens is None else tokens
    rng = np.random.default_rng(seed + 7919)
    return {
        "x": make_activations(rng, T, cfg.hidden, cfg.dtype, cfg.router),
        "attn_out": make_activations(rng, T, cfg.attn_dim, cfg.dtype, "random"),
        "w_router_attn": make_weight(rng, cfg.attn_n_groups, cfg.hidden,
                                     1.0 / np.sqrt(cfg.hidden), cfg.dtype),
        "w_o": make_weight(rng, cfg.hidden, cfg.attn_dim, 0.02, cfg.dtype),
    }


def make_attn_case(seed: int, tokens_q: int, tokens_k: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                   dtype: str = "bf16") -> Dict[str, np.ndarray]:
    """Host buffers for head-group-masked attention: q [T_q, H_q, d], k, v [T_k, H_kv, d] ~ N(0, 1)
    (the scale of normalised, RoPE-rotated projections), drawn independently."""
    rng = np.random.default_rng(seed + 611953)
    return {
        "q": make_activations(rng, tokens_q * n_q_heads, head_dim, dtype, "random").reshape(tokens_q, n_q_heads, head_dim),
        "k": make_activations(rng, tokens_k * n_kv_heads, head_dim, dtype, "random").reshape(tokens_k, n_kv_heads, head_dim),
        "v": make_activations(rng, tokens_k * n_kv_heads, head_dim, dtype, "random").reshape(tokens_k, n_kv_heads, head_dim),
    }


def make_pair_router(cfg: WideConfig, seed: int, rank: int = 16) -> Dict[str, np.ndarray]:
    """Bottleneck router weights W1 [D, r], W2 [r, 2*N_G] (Section 3.1, routing components)."""
    rng = np.random.default_rng(seed + 104729)
    return {
        "w1": make_weight(rng, cfg.hidden, rank, 1.0 / np.sqrt(cfg.hidden), cfg.dtype),
        "w2": make_weight(rng, rank, 2 * cfg.n_groups, 1.0 / np.sqrt(rank), cfg.dtype),
    }


def random_mask(seed: int, tokens: int, n_groups: int, k: int) -> np.ndarray:
    """A uniformly random {0,1}^[T, N_G] mask with exactly k ones per row (bool)."""
    rng = np.random.default_rng(seed + 15485863)
    m = np.zeros((tokens, n_groups), dtype=bool)
    for t in range(tokens):
        m[t, rng.permutation(n_groups)[:k]] = True
    return m


def bernoulli_mask(seed: int, tokens: int, n_groups: int, p: float) -> np.ndarray:
    """Independent Bernoulli(p) mask: variable number of active groups per token."""
    rng = np.random.default_rng(seed + 32452843)
    return rng.random((tokens, n_groups)) < p
