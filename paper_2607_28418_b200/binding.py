"""ctypes binding of libwide.so: the same entry points as include/wide.h, taking torch tensors.

Argument marshalling only -- every step of the path runs in the library's CUDA kernels.  Torch
is used for device memory and streams.  There is no fallback: if the shared library is missing
or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libwide.so")

OK = 0
BF16, F32 = 0, 1
ROUTE_TOPK, ROUTE_PAIR_ARGMAX = 0, 1
OP_ROUTE, OP_REORDER, OP_FFN, OP_OPROJ, OP_UNPERMUTE = 0, 1, 2, 3, 4
FLAG_NONE, FLAG_SIMT, FLAG_FORCE_PREFILL, FLAG_FORCE_DECODE, FLAG_INPUT_MASKED = 0, 1, 2, 4, 8
FLAG_KAXIS_GROUP, FLAG_KAXIS_OWNER, FLAG_REDUCE_BF16 = 16, 32, 64
FLAG_DECODE_TC = 128
DECODE_MAX_TOKENS = 64
DECODE_GEMV_MAX_TOKENS = 2
MAX_GROUPS = 256
ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = -1, -2, -3, -4, -5, -6

EXPORTS = ["wide_create", "wide_destroy", "wide_status", "wide_set_wait_limit_ns", "wide_profile_begin",
           "wide_profile_end", "wide_launch_count", "wide_selftest_wait", "wide_strerror",
           "wide_version", "wide_workspace_bytes", "wide_route", "wide_route_static", "wide_route_pair_prepared_bytes",
           "wide_route_pair_norm_workspace_bytes", "wide_route_pair_prepare", "wide_route_pair_norm", "wide_reorder",
           "wide_mask_slice", "wide_ffn_tp",
           "wide_ffn",
           "wide_oproj", "wide_attn", "wide_qproj", "wide_unpermute"]

_c_void_p, _c_int, _c_size_t, _c_uint = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t, ctypes.c_uint


class WideError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where} failed: {code} ({strerror(code)})")


_lib = None


def load_library() -> ctypes.CDLL:
    """Load libwide.so (built by ``python -m paper_2607_28418_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_28418_b200.build`; "
                           "there is no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    lib.wide_create.argtypes = [ctypes.POINTER(_c_void_p), _c_int]
    lib.wide_destroy.argtypes = [_c_void_p]
    lib.wide_status.argtypes = [_c_void_p, _c_void_p, ctypes.POINTER(_c_int)]
    lib.wide_set_wait_limit_ns.argtypes = [_c_void_p, ctypes.c_uint64]
    lib.wide_selftest_wait.argtypes = [_c_void_p, _c_void_p]
    lib.wide_profile_begin.argtypes = [_c_void_p, _c_int]
    lib.wide_profile_end.argtypes = [_c_void_p, _c_void_p, ctypes.c_char_p, _c_size_t]
    lib.wide_launch_count.argtypes = [_c_void_p, ctypes.POINTER(ctypes.c_ulonglong)]
    lib.wide_strerror.argtypes = [_c_int]
    lib.wide_strerror.restype = ctypes.c_char_p
    lib.wide_version.argtypes = []
    lib.wide_workspace_bytes.argtypes = [_c_int] * 7
    lib.wide_workspace_bytes.restype = _c_size_t
    lib.wide_route.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_void_p, _c_void_p,
                               _c_int, _c_int, _c_int, _c_int, _c_void_p, _c_void_p, _c_void_p, _c_void_p,
                               _c_size_t, _c_uint]
    lib.wide_route_static.argtypes = lib.wide_route.argtypes[:15] + [_c_uint]
    lib.wide_route_pair_prepared_bytes.argtypes = [_c_int] * 3
    lib.wide_route_pair_prepared_bytes.restype = _c_size_t
    lib.wide_route_pair_norm_workspace_bytes.argtypes = [_c_int] * 2
    lib.wide_route_pair_norm_workspace_bytes.restype = _c_size_t
    lib.wide_route_pair_prepare.argtypes = [_c_void_p] * 5 + [_c_int] * 3 + [_c_void_p, _c_size_t]
    lib.wide_route_pair_norm.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_void_p, _c_void_p, _c_int, _c_int,
                                         _c_void_p, ctypes.c_float, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_size_t]
    lib.wide_reorder.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int] + [_c_void_p] * 10
    lib.wide_mask_slice.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_int, _c_void_p]
    lib.wide_ffn.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_int, _c_int,
                             _c_int, _c_int, _c_int, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p,
                             _c_void_p, _c_int, _c_void_p, _c_size_t, _c_uint]
    lib.wide_ffn_tp.argtypes = [_c_void_p] * 6 + [_c_int] * 5 + [_c_void_p] * 6 + [_c_int, _c_int, _c_void_p, _c_size_t]
    lib.wide_oproj.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_int, _c_int,
                               _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_int,
                               _c_void_p, _c_size_t, _c_uint]
    lib.wide_attn.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_int,
                              _c_int, _c_int, _c_int, _c_void_p, _c_void_p, _c_void_p, _c_int, ctypes.c_float,
                              _c_void_p, _c_uint]
    lib.wide_qproj.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_int, _c_int,
                               _c_void_p, _c_void_p, _c_void_p, _c_uint]
    lib.wide_unpermute.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_int,
                                   _c_int, _c_int, _c_int, _c_void_p]
    for name in EXPORTS:
        if name not in ("wide_strerror", "wide_workspace_bytes", "wide_route_pair_prepared_bytes",
                        "wide_route_pair_norm_workspace_bytes"):
            getattr(lib, name).restype = _c_int
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().wide_strerror(code).decode()


def version() -> int:
    return load_library().wide_version()


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return _c_void_p(t.data_ptr())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise ValueError(f"unsupported dtype {t.dtype}")


def _stream() -> _c_void_p:
    return _c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code: int, where: str):
    if code != OK:
        raise WideError(code, where)


class Context:
    """Owns a wide_ctx for one device.  Scratch buffers are torch tensors cached per size."""

    def __init__(self, device: int = 0):
        self.lib = load_library()
        self.device = torch.device("cuda", device)
        h = _c_void_p()
        with torch.cuda.device(self.device):
            _check(self.lib.wide_create(ctypes.byref(h), device), "wide_create")
        self.handle = h
        self._ws: Dict[int, torch.Tensor] = {}

    def close(self):
        if self.handle:
            self.lib.wide_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace(self, nbytes: int, slot: int = 0) -> torch.Tensor:
        cur = self._ws.get(slot)
        if cur is None or cur.numel() < nbytes:
            cur = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=self.device)
            self._ws[slot] = cur
        return cur

    def status(self) -> int:
        v = _c_int(0)
        _check(self.lib.wide_status(self.handle, _stream(), ctypes.byref(v)), "wide_status")
        return v.value

    def set_wait_limit_ns(self, ns: int):
        _check(self.lib.wide_set_wait_limit_ns(self.handle, int(ns)), "wide_set_wait_limit_ns")

    def selftest_wait(self):
        """Enqueue the kernel whose only wait can never be satisfied (see wide_selftest_wait)."""
        _check(self.lib.wide_selftest_wait(self.handle, _stream()), "wide_selftest_wait")

    def profile_begin(self, max_records: int = 4096):
        _check(self.lib.wide_profile_begin(self.handle, max_records), "wide_profile_begin")

    def profile_end(self) -> Dict[str, Dict[str, float]]:
        """{kernel name: {"launches": n, "total_ms": t}} for everything launched since profile_begin."""
        buf = ctypes.create_string_buffer(8192)
        _check(self.lib.wide_profile_end(self.handle, _stream(), buf, len(buf)), "wide_profile_end")
        out = {}
        for line in buf.value.decode().splitlines():
            name, n, ms = line.split(",")
            out[name] = {"launches": int(n), "total_ms": float(ms)}
        return out

    def launch_count(self) -> int:
        v = ctypes.c_ulonglong(0)
        _check(self.lib.wide_launch_count(self.handle, ctypes.byref(v)), "wide_launch_count")
        return int(v.value)


def upload(a, dtype: str, device: Optional[torch.device] = None) -> torch.Tensor:
    """Host float32 array -> CUDA tensor of the workload dtype ("bf16": the values must already be
    bf16-representable, the upload is then exact; "fp32": as is)."""
    import numpy as np

    from . import synth
    device = device or torch.device("cuda", torch.cuda.current_device())
    if dtype == "bf16":
        bits = synth.to_bf16_bits(a)
        return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)


def workspace_bytes(op: int, dtype: int, tokens: int, hidden: int, inner: int, group: int, n_groups: int) -> int:
    return int(load_library().wide_workspace_bytes(op, dtype, tokens, hidden, inner, group, n_groups))


def wide_route(ctx: Context, x: torch.Tensor, w_router: torch.Tensor, n_groups: int, k: int = 0,
               mode: int = ROUTE_TOPK, w2: Optional[torch.Tensor] = None, rank: int = 0,
               k_per_token: Optional[torch.Tensor] = None, want_scores: bool = False,
               mask_bits: Optional[torch.Tensor] = None, flags: int = 0):
    """Returns (mask_bits int32 [T, W] holding the uint32 words, scores or None)."""
    T, D = x.shape
    W = (n_groups + 31) // 32
    if mask_bits is None:
        mask_bits = torch.empty((T, W), dtype=torch.int32, device=x.device)
    ncol = n_groups if mode == ROUTE_TOPK else 2 * n_groups
    scores = torch.empty((T, ncol), dtype=torch.float32, device=x.device) if want_scores else None
    nbytes = workspace_bytes(OP_ROUTE, _dtype_code(x), T, D, 0, 0, n_groups)
    ws = ctx.workspace(nbytes, slot=1)
    rc = ctx.lib.wide_route(ctx.handle, _stream(), _ptr(x), _dtype_code(x), T, D, _ptr(w_router), _ptr(w2), rank,
                            n_groups, mode, k, _ptr(k_per_token), _ptr(mask_bits), _ptr(scores), _ptr(ws),
                            ws.numel(), flags)
    _check(rc, "wide_route")
    return mask_bits, scores


def wide_route_pair_prepare(ctx: Context, w1: torch.Tensor, w2: torch.Tensor, norm_weight: Optional[torch.Tensor],
                            n_groups: int) -> torch.Tensor:
    """Once per weight set: the prepared buffer wide_route_pair_norm reads."""
    D, rank = w1.shape
    nbytes = int(ctx.lib.wide_route_pair_prepared_bytes(D, rank, n_groups))
    prepared = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=w1.device)
    rc = ctx.lib.wide_route_pair_prepare(ctx.handle, _stream(), _ptr(w1), _ptr(w2), _ptr(norm_weight), D, rank, n_groups,
                                         _ptr(prepared), prepared.numel())
    _check(rc, "wide_route_pair_prepare")
    return prepared


def wide_route_pair_norm(ctx: Context, x: torch.Tensor, w1: torch.Tensor, w2: torch.Tensor, norm_weight: Optional[torch.Tensor],
                         eps: float, prepared: torch.Tensor, n_groups: int, want_scores: bool = False,
                         mask_bits: Optional[torch.Tensor] = None):
    """Eq. 4 on RMSNorm(x): returns (mask_bits, logits of the normalised input or None)."""
    T, D = x.shape
    rank = w1.shape[1]
    if mask_bits is None:
        mask_bits = torch.empty((T, (n_groups + 31) // 32), dtype=torch.int32, device=x.device)
    scores = torch.empty((T, 2 * n_groups), dtype=torch.float32, device=x.device) if want_scores else None
    ws = ctx.workspace(int(ctx.lib.wide_route_pair_norm_workspace_bytes(T, rank)), slot=1)
    rc = ctx.lib.wide_route_pair_norm(ctx.handle, _stream(), _ptr(x), T, D, _ptr(w1), _ptr(w2), rank, n_groups,
                                      _ptr(norm_weight), float(eps), _ptr(prepared), _ptr(mask_bits), _ptr(scores), _ptr(ws),
                                      ws.numel())
    _check(rc, "wide_route_pair_norm")
    return mask_bits, scores


ROUTE_STATIC_BYTES = 2 << 20


def wide_route_static(ctx: Context, x: torch.Tensor, w_router: torch.Tensor, n_groups: int, k: int = 0,
                      mode: int = ROUTE_TOPK, w2: Optional[torch.Tensor] = None, rank: int = 0,
                      k_per_token: Optional[torch.Tensor] = None, scores: Optional[torch.Tensor] = None,
                      mask_bits: Optional[torch.Tensor] = None, flags: int = 0):
    """wide_route for callers that may not allocate: scratch is the library's fixed device array
    (problems beyond ROUTE_STATIC_BYTES of scratch are refused with ERR_WORKSPACE).  Pass
    preallocated ``mask_bits`` (and ``scores``) to keep the whole call allocation-free; calls that
    overlap on the GPU share the array and must be serialised by the caller."""
    T, D = x.shape
    if mask_bits is None:
        mask_bits = torch.empty((T, (n_groups + 31) // 32), dtype=torch.int32, device=x.device)
    rc = ctx.lib.wide_route_static(ctx.handle, _stream(), _ptr(x), _dtype_code(x), T, D, _ptr(w_router), _ptr(w2),
                                   rank, n_groups, mode, k, _ptr(k_per_token), _ptr(mask_bits), _ptr(scores), flags)
    _check(rc, "wide_route_static")
    return mask_bits, scores


def wide_reorder(ctx: Context, mask_bits: torch.Tensor, n_groups: int, tile_m: int = 128,
                 out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
    T = mask_bits.shape[0]
    n_tiles = (T + tile_m - 1) // tile_m
    dev = mask_bits.device
    if out is None:
        i32 = dict(dtype=torch.int32, device=dev)
        out = {
            "perm": torch.empty((n_groups, T), **i32),
            "counts": torch.empty((n_groups,), **i32),
            "tile_map": torch.empty((n_tiles, n_groups), dtype=torch.uint8, device=dev),
            "work_list": torch.empty((max(n_tiles * n_groups, 1), 2), **i32),
            "n_work": torch.empty((1,), **i32),
            "union_list": torch.empty((n_groups,), **i32),
            "n_union": torch.empty((1,), **i32),
            "offsets": torch.empty((n_groups + 1,), **i32),
            "token_order": torch.empty((T,), **i32),
            "token_rank": torch.empty((T,), **i32),
        }
    rc = ctx.lib.wide_reorder(ctx.handle, _stream(), _ptr(mask_bits), T, n_groups, tile_m, _ptr(out["perm"]),
                              _ptr(out["counts"]), _ptr(out["tile_map"]), _ptr(out["work_list"]),
                              _ptr(out["n_work"]), _ptr(out["union_list"]), _ptr(out["n_union"]),
                              _ptr(out["offsets"]), _ptr(out.get("token_order")), _ptr(out.get("token_rank")))
    _check(rc, "wide_reorder")
    return out


def group_range(n_groups: int, world: int, rank: int):
    """Groups [begin, end) owned by `rank` when n_groups are dealt to `world` ranks in contiguous,
    balanced ranges (the first n_groups % world ranks hold one group more)."""
    base, rem = divmod(n_groups, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)


def wide_mask_slice(ctx: Context, mask_bits: torch.Tensor, n_groups: int, group_begin: int, group_end: int,
                    out: Optional[torch.Tensor] = None) -> torch.Tensor:
    T = mask_bits.shape[0]
    if out is None:
        out = torch.empty((T, max(1, (group_end - group_begin + 31) // 32)), dtype=torch.int32, device=mask_bits.device)
    rc = ctx.lib.wide_mask_slice(ctx.handle, _stream(), _ptr(mask_bits), T, n_groups, group_begin, group_end, _ptr(out))
    _check(rc, "wide_mask_slice")
    return out


def wide_ffn_tp(ctx: Context, x: torch.Tensor, w_gate: torch.Tensor, w_up: torch.Tensor, w_down: torch.Tensor, group: int,
                mask_bits_local: torch.Tensor, meta: Dict[str, torch.Tensor], shard_ptrs, rows_per_rank: int):
    """One rank's group-sharded FFN part, added straight into the fp32 shards of the ranks that own
    the token rows.  ``shard_ptrs``: one device address per rank (ints), e.g. ``t.data_ptr()`` of a
    local tensor for this rank and the peer-mapped addresses of the others."""
    T, D = x.shape
    d_ff = w_gate.shape[0]
    world = len(shard_ptrs)
    table = (ctypes.c_void_p * world)(*[ctypes.c_void_p(int(p)) for p in shard_ptrs])
    nbytes = workspace_bytes(OP_FFN, BF16, T, D, d_ff, group, d_ff // group)
    ws = ctx.workspace(nbytes, slot=0)
    rc = ctx.lib.wide_ffn_tp(ctx.handle, _stream(), _ptr(x), _ptr(w_gate), _ptr(w_up), _ptr(w_down), _dtype_code(x), T, D,
                             d_ff, group, _ptr(mask_bits_local), _ptr(meta["perm"]), _ptr(meta["counts"]),
                             _ptr(meta.get("token_order")), _ptr(meta.get("token_rank")),
                             ctypes.cast(table, ctypes.c_void_p), world, rows_per_rank, _ptr(ws), ws.numel())
    _check(rc, "wide_ffn_tp")


def wide_ffn(ctx: Context, x: torch.Tensor, w_gate: torch.Tensor, w_up: torch.Tensor, w_down: torch.Tensor,
             group: int, mask_bits: torch.Tensor, meta: Optional[Dict[str, torch.Tensor]] = None,
             out_dtype: Optional[torch.dtype] = None, flags: int = 0, y: Optional[torch.Tensor] = None) -> torch.Tensor:
    T, D = x.shape
    d_ff = w_gate.shape[0]
    out_dtype = out_dtype or x.dtype
    if y is None:
        y = torch.empty((T, D), dtype=out_dtype, device=x.device)
    dt = _dtype_code(x)
    nbytes = workspace_bytes(OP_FFN, dt, T, D, d_ff, group, d_ff // group)
    ws = ctx.workspace(nbytes, slot=0)
    m = meta or {}
    rc = ctx.lib.wide_ffn(ctx.handle, _stream(), _ptr(x), _ptr(w_gate), _ptr(w_up), _ptr(w_down), dt, T, D, d_ff,
                          group, _ptr(mask_bits), _ptr(m.get("perm")), _ptr(m.get("counts")),
                          _ptr(m.get("token_order")), _ptr(m.get("token_rank")), _ptr(y), _dtype_code(y), _ptr(ws),
                          ws.numel(), flags)
    _check(rc, "wide_ffn")
    return y


def wide_oproj(ctx: Context, attn_out: torch.Tensor, w_o: torch.Tensor, group: int, mask_bits: torch.Tensor,
               meta: Optional[Dict[str, torch.Tensor]] = None, out_dtype: Optional[torch.dtype] = None,
               flags: int = 0, y: Optional[torch.Tensor] = None) -> torch.Tensor:
    T, K = attn_out.shape
    D = w_o.shape[0]
    out_dtype = out_dtype or attn_out.dtype
    if y is None:
        y = torch.empty((T, D), dtype=out_dtype, device=attn_out.device)
    dt = _dtype_code(attn_out)
    nbytes = workspace_bytes(OP_OPROJ, dt, T, D, K, group, K // group)
    ws = ctx.workspace(nbytes, slot=0)
    m = meta or {}
    rc = ctx.lib.wide_oproj(ctx.handle, _stream(), _ptr(attn_out), _ptr(w_o), dt, T, D, K, group, _ptr(mask_bits),
                            _ptr(m.get("perm")), _ptr(m.get("counts")), _ptr(m.get("token_order")),
                            _ptr(m.get("token_rank")), _ptr(y), _dtype_code(y), _ptr(ws), ws.numel(), flags)
    _check(rc, "wide_oproj")
    return y


def wide_attn(ctx: Context, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, n_q_heads: int, n_kv_heads: int,
              heads_per_group: int, meta: Optional[Dict[str, torch.Tensor]], causal: bool = True, scale: float = 0.0,
              flags: int = 0, o: Optional[torch.Tensor] = None, mask_bits: Optional[torch.Tensor] = None) -> torch.Tensor:
    """q [T_q, H_q*d], k/v [T_k, H_kv*d] bf16; meta = wide_reorder outputs of the attention mask
    (prefill form), mask_bits = the mask itself (decode form, a handful of query tokens)."""
    Tq, Tk = q.shape[0], k.shape[0]
    head_dim = q.shape[1] // n_q_heads
    if o is None:
        o = torch.empty_like(q)
    m = meta or {}
    rc = ctx.lib.wide_attn(ctx.handle, _stream(), _ptr(q), _ptr(k), _ptr(v), _dtype_code(q), Tq, Tk, n_q_heads,
                           n_kv_heads, head_dim, heads_per_group, _ptr(mask_bits), _ptr(m.get("perm")),
                           _ptr(m.get("counts")), 1 if causal else 0, float(scale), _ptr(o), flags)
    _check(rc, "wide_attn")
    return o


def wide_qproj(ctx: Context, x: torch.Tensor, w: torch.Tensor, group: int, meta: Dict[str, torch.Tensor],
               flags: int = 0, y: Optional[torch.Tensor] = None) -> torch.Tensor:
    """x [T, D], w [n_out, D] bf16; meta = wide_reorder outputs of the [T, n_out/group] mask."""
    T, D = x.shape
    n_out = w.shape[0]
    if y is None:
        y = torch.empty((T, n_out), dtype=x.dtype, device=x.device)
    rc = ctx.lib.wide_qproj(ctx.handle, _stream(), _ptr(x), _ptr(w), _dtype_code(x), T, D, n_out, group,
                            _ptr(meta["perm"]), _ptr(meta["counts"]), _ptr(y), flags)
    _check(rc, "wide_qproj")
    return y


def wide_unpermute(ctx: Context, src_packed: torch.Tensor, meta: Dict[str, torch.Tensor], tokens: int,
                   n_groups: int, group: int, dst: Optional[torch.Tensor] = None) -> torch.Tensor:
    if dst is None:
        dst = torch.empty((tokens, n_groups * group), dtype=src_packed.dtype, device=src_packed.device)
    rc = ctx.lib.wide_unpermute(ctx.handle, _stream(), _ptr(src_packed), _ptr(meta["perm"]), _ptr(meta["counts"]),
                                _ptr(meta["offsets"]), tokens, n_groups, group, src_packed.element_size(),
                                _ptr(dst))
    _check(rc, "wide_unpermute")
    return dst
