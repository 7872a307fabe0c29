"""CPU oracle for the WIDE hot path -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Plain, slow, fp64 numpy restatement of what the path computes, written from the
paper's definitions.  Only the tests, the smoke check and the benchmark's CPU
baseline may call it; the CUDA library never does and shares no code with it.

What follows which passage of the paper
---------------------------------------
route_scores          Routing components (Section 3.1): a linear map from the
                      activation to one score per group.  The paper's router is the
                      bottleneck pair form (Eq. 4, ``route_logits_pair`` +
                      ``mask_pair_argmax``); the single-linear + per-token top-k form
                      (``route_scores`` + ``mask_topk``) is the fixed-budget reading
                      "each token selects R groups" of Appendix A.
mask_pair_argmax      Eq. 4, inference branch: bit = [argmax over the class pair = 0].
route_logits_pair_norm  Eq. 4 applied to the RMSNorm of the hidden state (the router's input in a
                      pre-norm transformer block); rmsnorm is the textbook definition.
reorder               Eq. 6 / Algorithm 1 (per-column SortDesc, stable), the predicate
                      of Eq. 7-8 at level 0 (CTA tile), Appendix B's monotone shortcut.
cluster_tokens        not in the paper: one global token permutation (stable sort by a
                      hash of the mask row, the key is defined in the library header)
                      under which tiles of tokens share their active groups.
ffn                   Eq. 3 literally: (phi(X Wg^T) * (X Wu^T)) gated group-wise by the
                      mask, times Wd^T, with phi = SiLU.
oproj                 Eq. 2 / Eq. 10: (A gated group-wise) Wo^T.
unpermute/gather      the scatter epilogue of Algorithm 2 as a standalone step.
qproj                 the query projection under the head-group mask: (X Wq^T) gated
                      group-wise (N-axis gating of Section 3.3, Appendix A's N-axis form).
masked_attention      Eq. 1 with the head-group mask of Section 3.1 and the causal key
                      range of Algorithm 4 (delta = T_k - T_q): plain softmax attention
                      for every active (token, head group) pair, zeros elsewhere.  The
                      tiling, online softmax and pipelines of Algorithm 4 reach this
                      result up to rounding order, so the oracle is the definition.

Parity pins (tests/test_oracle_*.py): exact-rational brute force for scores and
top-k, closed-form one-hot routers, hand-worked reorder fixture, permutation /
monotonicity / boundary-tile invariants, dense-SwiGLU special case against a library
routine, brute-force single-group sums, additivity over disjoint masks (Eq. 10), the
per-token gather formulation of Appendix A, constant-weight closed forms; token
clustering: permutation / inverse / sortedness / stability / grouping properties and
two hand-expanded hash values; attention: a library attention routine for the all-ones
mask (MHA and GQA, with and without a key prefix), single-key / constant-V / zero-Q closed
forms, an explicit-loop brute force, key-shift invariance, exact zeros for inactive pairs.
"Parity to values printed in the paper": unpinned -- the paper prints no worked
numeric example for this path.

All floating point is fp64; inputs (fp32 or bf16-representable fp32) widen exactly.
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence, Union

import numpy as np

ArrayLike = Union[np.ndarray, Sequence]


def _f64(a: ArrayLike) -> np.ndarray:
    return np.asarray(a, dtype=np.float64)


# ----------------------------------------------------------------------------- routing
def route_scores(x: ArrayLike, w_router: ArrayLike) -> np.ndarray:
    """s[t, g] = sum_i x[t, i] * w_router[g, i]  (one linear layer, fp64)."""
    return _f64(x) @ _f64(w_router).T


def route_logits_pair(x: ArrayLike, w1: ArrayLike, w2: ArrayLike) -> np.ndarray:
    """Eq. 4: R = reshape(X W1 W2) in [T, N_G, 2]; W1 [D, r], W2 [r, 2 N_G]."""
    logits = (_f64(x) @ _f64(w1)) @ _f64(w2)
    return logits.reshape(logits.shape[0], -1, 2)


def rmsnorm(x: ArrayLike, weight: Optional[ArrayLike], eps: float) -> np.ndarray:
    """RMSNorm of the Llama backbones the paper prunes (Section 4.1): every row divided by the root
    of its mean square (plus eps), then scaled channel-wise by `weight` (None: no scaling)."""
    x = _f64(x)
    y = x / np.sqrt(np.mean(x * x, axis=1, keepdims=True) + float(eps))
    return y if weight is None else y * _f64(weight)[None, :]


def route_logits_pair_norm(x: ArrayLike, norm_weight: Optional[ArrayLike], eps: float, w1: ArrayLike,
                           w2: ArrayLike) -> np.ndarray:
    """Eq. 4 on the normalised activation: the router reads the layer's input after its RMSNorm
    (the router "maps the input activation", Section 3.1, and the pruned unit's input is the
    normalised hidden state), so R = reshape(RMSNorm(x) W1 W2)."""
    return route_logits_pair(rmsnorm(x, norm_weight, eps), w1, w2)


def mask_pair_argmax(logits_pair: np.ndarray) -> np.ndarray:
    """Eq. 4, inference: execute (bit 1) iff argmax over the pair is class 0.

    argmax returns the first maximal index, so a tie executes.
    """
    return np.argmax(logits_pair, axis=-1) == 0


def mask_topk(scores: np.ndarray, k: Union[int, ArrayLike]) -> np.ndarray:
    """Per token, mark the k groups with the largest score; equal scores -> lower index.

    ``k`` is a scalar or one integer per token (0 <= k <= N_G).
    """
    scores = _f64(scores)
    T, n_groups = scores.shape
    k_t = np.broadcast_to(np.asarray(k, dtype=np.int64), (T,))
    mask = np.zeros((T, n_groups), dtype=bool)
    for t in range(T):
        # total order: score descending, then group index ascending
        order = sorted(range(n_groups), key=lambda g: (-scores[t, g], g))
        mask[t, order[: int(k_t[t])]] = True
    return mask


def pack_mask_bits(mask: np.ndarray) -> np.ndarray:
    """Row-major bit packing: bit (g % 32) of word (g // 32) of row t is mask[t, g]."""
    mask = np.asarray(mask, dtype=bool)
    T, n_groups = mask.shape
    words = (n_groups + 31) // 32
    out = np.zeros((T, words), dtype=np.uint32)
    for g in range(n_groups):
        out[:, g // 32] |= mask[:, g].astype(np.uint32) << np.uint32(g % 32)
    return out


def unpack_mask_bits(bits: np.ndarray, n_groups: int) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint32)
    T = bits.shape[0]
    out = np.zeros((T, n_groups), dtype=bool)
    for g in range(n_groups):
        out[:, g] = (bits[:, g // 32] >> np.uint32(g % 32)) & 1
    return out


# ----------------------------------------------------------------------------- token clustering
def mask_key(words_row, n_groups: int) -> int:
    """Clustering key of one token (the definition stated in the library header): with at most 32
    groups the decisions for groups 0..7 as an integer (bit g = group g); with more groups the top
    8 bits of an FNV-1a style hash over its packed mask words (32-bit wrap-around arithmetic)."""
    if n_groups <= 32:
        return int(words_row[0]) & 0xFF
    h = 0x811C9DC5
    for w in words_row:
        h = ((h ^ int(w)) * 0x01000193) & 0xFFFFFFFF
    return h >> 24


def cluster_tokens(mask: np.ndarray) -> Dict[str, np.ndarray]:
    """One token permutation that makes tiles of tokens share their active groups (the global
    counterpart of the per-group sort of Eq. 6): tokens in a stable sort by mask_key, so tokens
    with identical masks are neighbours.  token_rank is the inverse of token_order."""
    bits = pack_mask_bits(mask)
    T = bits.shape[0]
    keys = [mask_key(bits[t], mask.shape[1]) for t in range(T)]
    order = sorted(range(T), key=lambda t: (keys[t], t))
    rank = [0] * T
    for p, t in enumerate(order):
        rank[t] = p
    return {"token_order": np.asarray(order, dtype=np.int32).reshape(T),
            "token_rank": np.asarray(rank, dtype=np.int32).reshape(T)}


# ----------------------------------------------------------------------------- reorder
def reorder(mask: np.ndarray, tile_m: int) -> Dict[str, np.ndarray]:
    """Mask reordering (Eq. 6, Algorithm 1) and the level-0 predicate (Eq. 7-8).

    For every routing column g the rows are sorted by mask value, descending and stable:
    active rows (ascending original index) first, then inactive rows (ascending).

    Returns
      perm        int32 [N_G, T]   perm[g, j] = original row at sorted position j  (I_{j,g})
      sorted_mask bool  [T, N_G]   sorted_mask[j, g] = mask[perm[g, j], g]          (M~)
      counts      int32 [N_G]      active rows per group
      tile_map    uint8 [n_tiles, N_G]  OR of sorted_mask over rows [m*BM, min((m+1)*BM, T))
      tile_any    uint8 [n_tiles, N_G]  OR of the *unsorted* mask over the same row range
      work_list   int32 [n_work, 2] active (tile, group) pairs, group-major, tile ascending
      n_work      int
      union_list  int32 [n_union]  groups with at least one active row, ascending
      n_union     int
      offsets     int32 [N_G + 1]  offsets[g] = sum_{g' < g} ceil(counts[g'] / BM) * BM
      token_order, token_rank  int32 [T]  see cluster_tokens
    """
    mask = np.asarray(mask, dtype=bool)
    T, n_groups = mask.shape
    n_tiles = (T + tile_m - 1) // tile_m
    perm = np.zeros((n_groups, T), dtype=np.int32)
    sorted_mask = np.zeros((T, n_groups), dtype=bool)
    counts = np.zeros(n_groups, dtype=np.int32)
    for g in range(n_groups):
        active = [t for t in range(T) if mask[t, g]]
        inactive = [t for t in range(T) if not mask[t, g]]
        perm[g, :] = active + inactive
        counts[g] = len(active)
        sorted_mask[:, g] = mask[perm[g, :], g]
    tile_map = np.zeros((n_tiles, n_groups), dtype=np.uint8)
    tile_any = np.zeros((n_tiles, n_groups), dtype=np.uint8)
    for m in range(n_tiles):
        lo, hi = m * tile_m, min((m + 1) * tile_m, T)
        for g in range(n_groups):
            tile_map[m, g] = 1 if sorted_mask[lo:hi, g].any() else 0
            tile_any[m, g] = 1 if mask[lo:hi, g].any() else 0
    work = [(m, g) for g in range(n_groups) for m in range(n_tiles) if tile_map[m, g]]
    union = [g for g in range(n_groups) if counts[g] > 0]
    offsets = np.zeros(n_groups + 1, dtype=np.int32)
    for g in range(n_groups):
        offsets[g + 1] = offsets[g] + ((int(counts[g]) + tile_m - 1) // tile_m) * tile_m
    clustered = cluster_tokens(mask)
    return {
        "token_order": clustered["token_order"],
        "token_rank": clustered["token_rank"],
        "perm": perm,
        "sorted_mask": sorted_mask,
        "counts": counts,
        "tile_map": tile_map,
        "tile_any": tile_any,
        "work_list": np.asarray(work, dtype=np.int32).reshape(-1, 2),
        "n_work": len(work),
        "union_list": np.asarray(union, dtype=np.int32),
        "n_union": len(union),
        "offsets": offsets,
    }


# ----------------------------------------------------------------------------- FFN / O-proj
def expand_group_mask(mask: np.ndarray, group: int) -> np.ndarray:
    """[T, N_G] -> [T, N_G * G]: every group bit repeated over its G channels."""
    return np.repeat(np.asarray(mask, dtype=bool), group, axis=1)


def silu(a: np.ndarray) -> np.ndarray:
    """phi(a) = a * sigmoid(a) = a / (1 + exp(-a))."""
    a = _f64(a)
    return a / (1.0 + np.exp(-a))


def ffn_hidden(x: ArrayLike, w_gate: ArrayLike, w_up: ArrayLike, mask: np.ndarray,
               group: int) -> np.ndarray:
    """Inner term of Eq. 3: (phi(X Wg^T) * (X Wu^T)) gated by the group mask -> [T, D']."""
    x = _f64(x)
    h = silu(x @ _f64(w_gate).T) * (x @ _f64(w_up).T)
    return np.where(expand_group_mask(mask, group), h, 0.0)


def ffn(x: ArrayLike, w_gate: ArrayLike, w_up: ArrayLike, w_down: ArrayLike,
        mask: np.ndarray, group: int) -> np.ndarray:
    """Eq. 3: X' = ((phi(X Wg^T) * (X Wu^T)) (.)_G M) Wd^T  -> [T, D], fp64."""
    return ffn_hidden(x, w_gate, w_up, mask, group) @ _f64(w_down).T


def oproj(attn_out: ArrayLike, w_o: ArrayLike, mask: np.ndarray, group: int) -> np.ndarray:
    """Eq. 2 (second line) / Eq. 10: X' = (Attn (.)_G M) Wo^T, channels head-major."""
    a = np.where(expand_group_mask(mask, group), _f64(attn_out), 0.0)
    return a @ _f64(w_o).T


# ----------------------------------------------------------------------------- gather / scatter
def qproj(x: ArrayLike, w: ArrayLike, mask: np.ndarray, group: int) -> np.ndarray:
    """Routed query projection (Section 3.1; the N-axis case of Section 3.3): the output channels of
    group g are computed for the tokens that selected g and are zero for the others,
    y = (x W^T) gated group-wise by the mask.  x [T, D], w [n_out, D], mask [T, n_out/group]."""
    return (_f64(x) @ _f64(w).T) * expand_group_mask(mask, group)


def masked_attention(q: ArrayLike, k: ArrayLike, v: ArrayLike, mask: np.ndarray, heads_per_group: int,
                     causal: bool = True, scale: Optional[float] = None) -> np.ndarray:
    """Head-group-masked softmax attention (Eq. 1, Section 3.1; key range of Algorithm 4).

    q [T_q, H_q, d]; k, v [T_k, H_kv, d] (H_q a multiple of H_kv: query head h reads KV head
    h // (H_q / H_kv)); mask [T_q, N_G] bool with routing group g = heads [g*hpg, (g+1)*hpg).
    For an active pair (t, g) and each head h of g:
        o[t, h] = sum_j softmax_j(scale * q[t, h] . k[j, h_kv]) * v[j, h_kv]
    over keys j <= t + (T_k - T_q) when causal, all keys otherwise; scale defaults to
    1/sqrt(d).  Inactive pairs give exact zeros, and so does a query that sees no key at all
    (t + T_k - T_q < 0; Algorithm 4 leaves such a row's state at its zero initial value).
    """
    q, k, v = _f64(q), _f64(k), _f64(v)
    t_q, h_q, d = q.shape
    t_k, h_kv, _ = k.shape
    rep = h_q // h_kv
    delta = t_k - t_q
    sc = 1.0 / np.sqrt(d) if scale is None else float(scale)
    out = np.zeros((t_q, h_q, d))
    key_pos = np.arange(t_k)[None, :]
    qry_pos = np.arange(t_q)[:, None] + delta
    for h in range(h_q):
        rows = np.nonzero(mask[:, h // heads_per_group])[0]
        if rows.size == 0:
            continue
        s = sc * (q[rows, h, :] @ k[:, h // rep, :].T)            # [rows, T_k]
        if causal:
            seen = qry_pos[rows, 0] >= 0          # a query before the first key sees nothing: zeros
            rows, s = rows[seen], s[seen]
            s = np.where(key_pos <= qry_pos[rows], s, -np.inf)
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        p /= p.sum(axis=1, keepdims=True)
        out[rows, h, :] = p @ v[:, h // rep, :]
    return out


def gather_packed(dense: np.ndarray, perm: np.ndarray, counts: np.ndarray,
                  offsets: np.ndarray, group: int) -> np.ndarray:
    """Dense [T, N_G*G] -> packed-sorted [offsets[N_G], G]: row offsets[g]+j holds the
    group-g slice of original row perm[g, j] for j < counts[g]; padding rows are zero."""
    dense = np.asarray(dense)
    n_groups = perm.shape[0]
    out = np.zeros((int(offsets[n_groups]), group), dtype=dense.dtype)
    for g in range(n_groups):
        for j in range(int(counts[g])):
            out[int(offsets[g]) + j, :] = dense[perm[g, j], g * group:(g + 1) * group]
    return out


def unpermute(src_packed: np.ndarray, perm: np.ndarray, counts: np.ndarray,
              offsets: np.ndarray, tokens: int, group: int) -> np.ndarray:
    """Scatter epilogue as its own step: dst[perm[g, j], g*G:(g+1)*G] = src[offsets[g]+j]
    for j < counts[g]; every other element of dst is zero."""
    src_packed = np.asarray(src_packed)
    n_groups = perm.shape[0]
    dst = np.zeros((tokens, n_groups * group), dtype=src_packed.dtype)
    for g in range(n_groups):
        for j in range(int(counts[g])):
            dst[perm[g, j], g * group:(g + 1) * group] = src_packed[int(offsets[g]) + j, :]
    return dst


# ----------------------------------------------------------------------------- whole path
def layer_ffn(x: ArrayLike, w_router: ArrayLike, w_gate: ArrayLike, w_up: ArrayLike,
              w_down: ArrayLike, group: int, k: Union[int, ArrayLike],
              tile_m: int = 128) -> Dict[str, np.ndarray]:
    """route -> top-k mask -> reorder -> masked FFN, every intermediate returned."""
    scores = route_scores(x, w_router)
    mask = mask_topk(scores, k)
    meta = reorder(mask, tile_m)
    y = ffn(x, w_gate, w_up, w_down, mask, group)
    out = {"scores": scores, "mask": mask, "mask_bits": pack_mask_bits(mask), "y": y}
    out.update(meta)
    return out
