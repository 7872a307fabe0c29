#!/usr/bin/env python
"""Benchmark of the WIDE hot path (route -> reorder -> masked SwiGLU FFN) on synthetic
Llama-shaped layers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload llama7b_prefill|llama8b_prefill|llama13b_layer|llama8b_decode]
                    [--batch B] [--router random|clustered|clustered_corr] [--k K] [--group G]

One step = one pass of the whole path over one batch of tokens.  Rank 0 prints one JSON line.
With N > 1 (torchrun) every rank runs its own token shard with replicated weights and no
data-path collective (weak scaling); the timed region is bracketed by a barrier and the elapsed
time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_28418_b200 import synth  # noqa: E402

METRIC = "masked-layer tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}
NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}   # the part's data-sheet figures (dense)
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the committed ncu summaries,
# keyed by (kernel, workload) -> (bytes, the summary under profiles/ it was read from).
NCU_TRAFFIC_BYTES = {
    ("prefill_gateup", "llama7b_prefill"): (292.3e6, "profiles/prefill_llama7b_gateup_down_kernels.md"),
    ("prefill_down", "llama7b_prefill"): (140.1e6, "profiles/prefill_llama7b_gateup_down_kernels.md"),
    # decode: captured at batch 8 (union 111 groups, 357.3 MB); traffic is proportional to the union
    ("decode_ffn_fused", "llama8b_decode"): (357.3e6 / 111, "profiles/decode_llama8b_batch8_fused_kernel.md"),
    # captured at batch 1 (union 56 groups, 180.4 MB)
    ("decode_ffn_gemv", "llama8b_decode"): (180.4e6 / 56, "profiles/decode_llama8b_batch1_gemv_kernel.md"),
}


def ncu_traffic(kernel, workload, scale=1.0):
    """(traffic bytes per launch or None, source file or None)."""
    hit = NCU_TRAFFIC_BYTES.get((kernel, workload))
    return (hit[0] * scale, hit[1]) if hit else (None, None)


def roofline_record(kernel, bound, achieved, peaks, traffic=None, traffic_source=None, **extra):
    """One roofline object: the fraction against the measured peak of this machine (the headline
    `frac`) and against the part's nominal figure."""
    key, unit = ("hbm_gbs", "GB/s") if bound == "hbm" else ("bf16_tflops", "TFLOP/s")
    rec = {"kernel": kernel, "bound": bound, "achieved": achieved, "peak": peaks[key], "unit": unit,
           "frac": achieved / peaks[key], "frac_measured": achieved / peaks[key],
           "peak_nominal": NOMINAL_PEAKS[key], "frac_nominal": achieved / NOMINAL_PEAKS[key],
           "traffic": traffic, "traffic_source": traffic_source, "peak_source": peaks["source"]}
    rec.update(extra)
    return rec


def weight_copies(cfg, n_mats, flush_l2):
    """Decode steps rotate over this many identical copies of the weights (> 4x L2 in all), so every
    step streams its weights from HBM; prefill weights are larger than L2 by themselves."""
    if cfg.tokens > 64 or flush_l2:
        return 1
    return max(2, -(-(640 << 20) // (n_mats * cfg.d_ff * cfg.hidden * 2)))


def config_record(cfg, op, world, flush_l2=False):
    """The workload description both arms print (same keys, same values).  `cfg` describes the
    operation timed: for the attention-half operations d_ff / group / k are the attention
    dimension, its group size and its budget."""
    n_mats = 3 if op == "ffn" else 1
    weights_mb = n_mats * cfg.d_ff * cfg.hidden * 2 / 1e6
    n_copies = weight_copies(cfg, n_mats, flush_l2)
    l2 = ("flushed between steps" if flush_l2 else
          "weights rotate over %d copies (%.0f MB), every step streams from HBM" % (n_copies, n_copies * weights_mb)
          if n_copies > 1 else "inputs larger than L2 (weights %.0f MB)" % weights_mb)
    return {"workload": cfg.name, "op": op, "tokens_per_gpu": cfg.tokens, "hidden": cfg.hidden, "d_ff": cfg.d_ff,
            "group": cfg.group, "n_groups": cfg.n_groups, "k": cfg.k, "router": cfg.router,
            "parallelism": f"token-sharded x{world}, weights replicated, no collective", "l2": l2}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return dict(FALLBACK_PEAKS)


# ------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------- workload
def make_config(args) -> synth.WideConfig:
    cfg = synth.CONFIGS[args.workload]
    kw = {}
    if args.batch:
        kw["tokens"] = args.batch
    if args.router:
        kw["router"] = args.router
    if args.group:
        kw["group"] = args.group
        kw["k"] = (cfg.d_ff // args.group) * cfg.k // cfg.n_groups
    if args.k is not None:
        kw["k"] = args.k
    return cfg.with_(**kw) if kw else cfg


def aggregate(units_per_rank: float, steps: int, elapsed_ms_max: float, world: int) -> float:
    """Whole-job throughput: units processed by all ranks / (max-over-ranks time)."""
    return units_per_rank * world * steps / (elapsed_ms_max * 1e-3)


def reduce_max_ms(ms: float, world: int, device=None) -> float:
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def flops_ffn_active(cfg, oproj: bool = False) -> float:
    return (2.0 if oproj else 6.0) * cfg.tokens * cfg.k * cfg.group * cfg.hidden


# ------------------------------------------------------------------------------- reference arm
def oracle_sample_step(case, cfg, sample_tokens):
    from oracle import wide_oracle as wo
    return wo.layer_ffn(case["x"][:sample_tokens], case["w_router"], case["w_gate"], case["w_up"], case["w_down"],
                        cfg.group, cfg.k, cfg.tile_m)


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def time_oracle(case, cfg, sample_tokens, steps, warmup):
    for _ in range(warmup):
        oracle_sample_step(case, cfg, sample_tokens)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_sample_step(case, cfg, sample_tokens)
    dt = time.perf_counter() - t0
    return sample_tokens * steps / dt, dt / steps * 1e3


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = make_config(args)
    case = synth.make_ffn_case(cfg, 0, tokens=min(cfg.tokens, args.oracle_tokens))
    sample = min(cfg.tokens, args.oracle_tokens)
    steps = max(1, args.steps)
    warmup = max(3, args.warmup)
    value, ms = time_oracle(case, cfg, sample, steps, warmup)
    cores = blas_threads()
    world = int(os.environ.get("WORLD_SIZE", "1"))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_record(cfg, args.op, world, args.flush_l2),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                         "sample": f"each step = the first {sample} of {cfg.tokens} tokens through route, top-k, "
                                   "reorder and the masked FFN in fp64 numpy"},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------- extra records
def graph_of(torch, fn):
    """Capture one call of fn (library calls only enqueue kernels on the current stream)."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        fn()
    torch.cuda.current_stream().wait_stream(side)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g.replay


def event_ms(torch, fn, reps):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def sustained_record(torch, run_step, ms_hint, tokens, flops_ffn, peaks, gpu_index, seconds=2.0):
    """The same step graph replayed back to back for `seconds`: what the path does once the part
    has settled under its power cap, with the median SM clock seen meanwhile.  The fraction counts
    the FFN's active FLOPs against the whole step (routing included), so it is a lower bound."""
    reps = max(10, int(seconds / (ms_hint * 1e-3)))
    sampler = ClockSampler(gpu_index)
    sampler.start()
    ms = event_ms(torch, run_step, reps)
    clocks = sampler.stop()
    tfl = flops_ffn / (ms * 1e-3) / 1e12
    peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    return {"seconds": round(reps * ms * 1e-3, 3), "replays": reps, "ms_per_step": ms, "value": tokens / (ms * 1e-3),
            "unit": "tokens/s", "clocks": clocks, "ffn_active_tflops_over_step": tfl, "peak_sustained": peak,
            "frac_of_sustained_peak": tfl / peak, "frac_of_nominal_peak": tfl / NOMINAL_PEAKS["bf16_tflops"]}


def cublas_dense_context(torch, d, reps=10):
    """Context only, not on the path: the dense SwiGLU FFN of the same shape through torch.matmul
    (cuBLAS), the paper's own dense baseline for its kernel speed-ups."""
    x, wg, wu, wd = d["x"], d["w_gate"], d["w_up"], d["w_down"]

    def dense():
        return (torch.nn.functional.silu(x @ wg.t()) * (x @ wu.t())) @ wd.t()
    for _ in range(3):
        dense()
    ms = event_ms(torch, dense, reps)
    return {"ms": ms, "what": "silu(x Wg^T) * (x Wu^T) then Wd^T through torch.matmul (cuBLAS), bf16; "
                              "off the path, quoted beside the speed-up over our own dense run",
            "dense_tflops": 6.0 * x.shape[0] * wg.shape[0] * x.shape[1] / (ms * 1e-3) / 1e12}


def decode_sweep(torch, binding, ctx, peaks, gpu_index, batches=(1, 8, 16, 32, 64), replays=300, flags=0):
    """Llama-3-8B-shaped decode FFN (hidden 4096, d_ff 14336, 112 groups of 128, top-56, random
    router) at each batch size: the FFN call replayed as a graph over two rotating copies of the
    weights (704 MB > 4x L2, so every replay streams from HBM), and the whole step (route + FFN)."""
    cfg = synth.CONFIGS["llama8b_decode"].with_(tokens=64)
    case = synth.make_ffn_case(cfg, 0)
    d = {k: binding.upload(v, "bf16") for k, v in case.items()}
    wsets = [{k: d[k] for k in ("w_gate", "w_up", "w_down")}]
    wsets.append({k: v.clone() for k, v in wsets[0].items()})
    per_group = cfg.group * cfg.hidden * 2
    sampler = ClockSampler(gpu_index)
    sampler.start()
    out = []
    for B in batches:
        x = d["x"][:B].contiguous()
        bits = torch.empty((B, (cfg.n_groups + 31) // 32), dtype=torch.int32, device=x.device)
        y = torch.empty((B, cfg.hidden), dtype=torch.bfloat16, device=x.device)
        binding.wide_route(ctx, x, d["w_router"], cfg.n_groups, cfg.k, mask_bits=bits)

        def ffn(c):
            w = wsets[c]
            binding.wide_ffn(ctx, x, w["w_gate"], w["w_up"], w["w_down"], cfg.group, bits, None, y=y, flags=flags)

        def whole(c):
            binding.wide_route(ctx, x, d["w_router"], cfg.n_groups, cfg.k, mask_bits=bits)
            ffn(c)
        for c in range(2):
            ffn(c)
        g_ffn = [graph_of(torch, lambda c=c: ffn(c)) for c in range(2)]
        g_all = [graph_of(torch, lambda c=c: whole(c)) for c in range(2)]
        state = {"i": 0}

        def rot(graphs):
            def run():
                graphs[state["i"] & 1]()
                state["i"] += 1
            return run
        event_ms(torch, rot(g_ffn), 6)
        ffn_ms = event_ms(torch, rot(g_ffn), replays)
        step_ms = event_ms(torch, rot(g_all), replays)
        union_words = np.bitwise_or.reduce(bits.cpu().numpy().view(np.uint32), axis=0)
        n_union = sum(bin(int(w)).count("1") for w in union_words)
        gbs = 3.0 * n_union * per_group / (ffn_ms * 1e-3) / 1e9
        out.append({"batch": B, "ffn_ms": ffn_ms, "step_ms": step_ms, "n_union": n_union, "achieved_gbs": gbs,
                    "frac": gbs / peaks["hbm_gbs"], "frac_nominal": gbs / NOMINAL_PEAKS["hbm_gbs"],
                    "tokens_per_s": B / (step_ms * 1e-3)})
    if ctx.status() != 0:
        raise RuntimeError("device status word set during the decode sweep")
    clocks = sampler.stop()
    return {"workload": "llama8b_decode", "router": "random", "k": cfg.k, "n_groups": cfg.n_groups,
            "bytes": "union groups x 3 x group x hidden x 2 B (gate, up, down weights)", "peak": peaks["hbm_gbs"],
            "peak_source": peaks["source"], "replays": replays, "clocks": clocks, "points": out}


def oproj_13b_record(torch, binding, ctx, peaks, replays=50):
    """Llama-2-13B-shaped head-group-masked output projection (T = 4096, 40 heads of 128 in 10 groups,
    top-5): the wide_oproj call alone as a graph, with the library's own choice of K-axis kernel and
    with the owner-computes kernel forced, and with every group active (the dense run of the same
    call)."""
    cfg = synth.CONFIGS["llama13b_layer"]
    case = synth.make_oproj_case(cfg, 0)
    d = {k: binding.upload(v, "bf16") for k, v in case.items()}
    T, NG, G = cfg.tokens, cfg.attn_n_groups, cfg.attn_group
    y = torch.empty((T, cfg.hidden), dtype=torch.bfloat16, device=d["x"].device)
    out = {"workload": "llama13b_layer", "op": "oproj", "tokens": T, "n_groups": NG, "group": G}
    for k in (cfg.attn_k, NG):
        bits, _ = binding.wide_route(ctx, d["x"], d["w_router_attn"], NG, k)
        meta = binding.wide_reorder(ctx, bits, NG, 128)
        for name, flags in (("auto", 0), ("owner", binding.FLAG_KAXIS_OWNER)):
            def call():
                binding.wide_oproj(ctx, d["attn_out"], d["w_o"], G, bits, meta, y=y, flags=flags)
            for _ in range(3):
                call()
            g = graph_of(torch, call)
            g()
            ms = event_ms(torch, g, replays)
            tag = f"k{k}_{name}"
            out[tag + "_ms"] = ms
            if k == cfg.attn_k:
                tfl = 2.0 * T * k * G * cfg.hidden / (ms * 1e-3) / 1e12
                out[tag + "_active_tflops"] = tfl
                out[tag + "_frac_of_bf16_peak"] = tfl / peaks["bf16_tflops"]
    if ctx.status() != 0:
        raise RuntimeError("device status word set during the O-projection record")
    out["speedup_vs_all_groups_active"] = out[f"k{NG}_auto_ms"] / out[f"k{cfg.attn_k}_auto_ms"]
    out["ideal"] = NG / cfg.attn_k
    return out


def attn_13b_record(torch, binding, ctx, peaks, replays=30):
    """Llama-2-13B-shaped head-group-masked causal attention, prefill (one sequence of 4096 positions,
    40 heads of 128 in 10 groups, top-5): the wide_attn call alone as a graph; FLOPs counted per
    active (token, head) pair over its visible keys."""
    cfg = synth.CONFIGS["llama13b_layer"]
    T, hd = cfg.tokens, 128
    H, hpg, NG, k = cfg.attn_dim // hd, cfg.attn_group // hd, cfg.attn_n_groups, cfg.attn_k
    oc = synth.make_oproj_case(cfg, 0)
    ac = synth.make_attn_case(0, T, T, H, H, hd)
    x, wr = binding.upload(oc["x"], "bf16"), binding.upload(oc["w_router_attn"], "bf16")
    q, kk, v = (binding.upload(ac[n].reshape(T, H * hd), "bf16") for n in ("q", "k", "v"))
    bits, _ = binding.wide_route(ctx, x, wr, NG, k)
    meta = binding.wide_reorder(ctx, bits, NG, 128)
    o = torch.empty_like(q)

    def call():
        binding.wide_attn(ctx, q, kk, v, H, H, hpg, meta, causal=True, o=o)
    for _ in range(3):
        call()
    g = graph_of(torch, call)
    g()
    ms = event_ms(torch, g, replays)
    if ctx.status() != 0:
        raise RuntimeError("device status word set during the attention record")
    mask = np.unpackbits(bits.cpu().numpy().view(np.uint8), axis=1, bitorder="little")[:, :NG].astype(bool)
    flops = float((mask.sum(axis=1) * hpg * 4.0 * hd * (np.arange(T) + 1.0)).sum())
    tfl = flops / (ms * 1e-3) / 1e12
    return {"workload": "llama13b_layer", "op": "attn", "tokens": T, "heads": H, "head_dim": hd, "n_groups": NG, "k": k,
            "ms": ms, "active_gflop": flops / 1e9, "active_tflops": tfl, "frac_of_bf16_peak": tfl / peaks["bf16_tflops"],
            "frac_of_nominal_peak": tfl / NOMINAL_PEAKS["bf16_tflops"]}


# ------------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2607_28418_b200 import binding
    to_dev = binding.upload

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    cfg = make_config(args)
    peaks = load_peaks()
    ctx = binding.Context(local)
    qproj = args.op == "qproj"
    oproj = args.op == "oproj" or qproj    # both run on the attention half: one GEMM, attention groups
    if oproj:
        case = synth.make_oproj_case(cfg, 1000 * rank)  # every rank its own token shard
        case["w_router"] = case.pop("w_router_attn")
        if qproj:   # routed query projection: W_q [H*d, D], output [T, H*d]
            case.pop("w_o")
            case.pop("attn_out")
            case["w_q"] = synth.make_weight(np.random.default_rng(1000 * rank + 17), cfg.attn_dim, cfg.hidden, 0.02, cfg.dtype)
        cfg = cfg.with_(d_ff=cfg.attn_dim, group=cfg.attn_group, k=cfg.attn_k)  # the op's inner dim / groups
    else:
        case = synth.make_ffn_case(cfg, 1000 * rank)
    d = {k: to_dev(v, cfg.dtype) for k, v in case.items()}
    T, NG = cfg.tokens, cfg.n_groups
    W = (NG + 31) // 32
    bits = torch.empty((T, W), dtype=torch.int32, device=dev)
    out_dim = cfg.d_ff if qproj else cfg.hidden
    y = torch.empty((T, out_dim), dtype=torch.bfloat16, device=dev)
    meta = None
    decode = T <= binding.DECODE_MAX_TOKENS

    xbuf = [d["x"], torch.empty_like(d["x"])]
    ybuf = [y, torch.empty_like(y)]

    # Decode: successive steps stand for successive layers of a model, each with its own weights.
    # The FFN weights rotate over several identical copies (> 4x L2 in total), so every step streams
    # its weights from HBM although the launches run back to back without an L2 flush in between.
    n_copies = weight_copies(cfg, 1 if oproj else 3, args.flush_l2)
    wkeys = ("w_q",) if qproj else ("w_o",) if oproj else ("w_gate", "w_up", "w_down")
    wsets = [{k: d[k] for k in wkeys}]
    for _ in range(n_copies - 1):
        wsets.append({k: d[k].clone() for k in wkeys})

    kflags = {"auto": 0, "group": binding.FLAG_KAXIS_GROUP, "owner": binding.FLAG_KAXIS_OWNER}[args.kaxis]
    dflags = binding.FLAG_DECODE_TC if args.decode_tc else 0
    if args.reduce_bf16:
        kflags |= binding.FLAG_REDUCE_BF16

    def main_op(x_in, w, y_out):
        if qproj:
            binding.wide_qproj(ctx, x_in, w["w_q"], cfg.group, meta, y=y_out)
        elif oproj:
            binding.wide_oproj(ctx, d["attn_out"], w["w_o"], cfg.group, bits, meta, y=y_out,
                               flags=(binding.FLAG_INPUT_MASKED if args.premasked else 0) | (dflags if decode else kflags))
        else:
            binding.wide_ffn(ctx, x_in, w["w_gate"], w["w_up"], w["w_down"], cfg.group, bits, meta, y=y_out,
                             flags=dflags if decode else kflags)
    calls = {"n": 0}

    def step(k=cfg.k, slot=0, copy=None):
        nonlocal meta
        if copy is None:
            copy = calls["n"] % n_copies
            calls["n"] += 1
        w = wsets[copy]
        x_in, y_out = xbuf[slot], ybuf[slot]
        binding.wide_route(ctx, x_in, d["w_router"], NG, k, mask_bits=bits)
        if not decode:
            meta = binding.wide_reorder(ctx, bits, NG, 128, out=meta)
        main_op(x_in, w, y_out)

    def rotating(make):
        """One graph per weight copy; successive calls replay them in turn."""
        runs = [graphed(lambda c=c: make(c)) for c in range(n_copies)]
        state = {"i": 0}

        def run():
            runs[state["i"] % n_copies]()
            state["i"] += 1
        return run

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sync_all()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        sync_all()
        return reduce_max_ms(e0.elapsed_time(e1), world, dev)

    def graphed(fn):
        """Capture one call of fn into a CUDA graph (the library only enqueues kernels and memsets
        on the current stream, so a whole step replays as one launch)."""
        if args.no_graph:
            return fn
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g.replay

    flush = None
    if args.flush_l2:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    for _ in range(max(3, args.warmup)):
        step()
    if ctx.status() != 0:
        raise RuntimeError("device status word set during warm-up")
    if args.premasked and args.op == "oproj":
        # the attention output as wide_attn leaves it: zeros for inactive (token, group) pairs
        # (x and hence the mask are the same in every step)
        m = (bits.view(torch.int32)[:, :, None] >> torch.arange(32, device=dev, dtype=torch.int32)) & 1
        m = m.reshape(T, -1)[:, :NG].to(torch.bfloat16).repeat_interleave(cfg.group, dim=1)
        d["attn_out"] = (d["attn_out"] * m).contiguous()
    run_step = rotating(lambda c: step(copy=c))
    for _ in range(n_copies):
        run_step()

    # ---- timed region: K steps
    sampler = ClockSampler(local)
    sampler.start()
    if flush is None:
        ms_total = timed(run_step, args.steps)
    else:
        # flush L2 between steps (outside the timed brackets), time each step by itself
        ms_total = 0.0
        for _ in range(args.steps):
            flush.zero_()
            ms_total += timed(run_step, 1)
    if ctx.status() != 0:
        raise RuntimeError("device status word set during the timed region")
    value = aggregate(T, args.steps, ms_total, world)

    # ---- the FFN call alone, replayed as a graph: at decode sizes the host cannot enqueue as fast
    # as the GPU runs, so event pairs recorded around direct launches would include idle time
    run_ffn = rotating(lambda c: main_op(xbuf[0], wsets[c], ybuf[0]))
    for _ in range(n_copies):
        run_ffn()
    if flush is None:
        ffn_graph_ms = timed(run_ffn, args.steps) / args.steps
    else:
        ffn_graph_ms = 0.0
        for _ in range(args.steps):
            flush.zero_()
            ffn_graph_ms += timed(run_ffn, 1) / args.steps

    # ---- the same K steps again, every kernel bracketed by the library's own event pairs
    launches0 = ctx.launch_count()
    ctx.profile_begin(64 * args.steps + 64)
    for _ in range(args.steps):
        if flush is not None:
            flush.zero_()
        step()
    prof = ctx.profile_end()
    launches = ctx.launch_count() - launches0

    # ---- end to end: pinned host input -> device, whole path, result -> host, every step;
    # double-buffered over three streams so the copies of neighbouring steps overlap the compute
    x_host = torch.from_numpy(synth.to_bf16_bits(case["x"]).view(np.int16)).view(torch.bfloat16).pin_memory()
    y_host = [torch.empty((T, out_dim), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    s_in, s_run, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev = {n: [torch.cuda.Event(), torch.cuda.Event()] for n in ("in", "run", "out")}

    def e2e_loop(steps):
        cur = torch.cuda.current_stream()
        for st in (s_in, s_run, s_out):
            st.wait_stream(cur)
        for i in range(steps):
            b = i % 2
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev["run"][b])      # step i-2 has consumed xbuf[b]
                xbuf[b].copy_(x_host, non_blocking=True)
                ev["in"][b].record()
            with torch.cuda.stream(s_run):
                s_run.wait_event(ev["in"][b])
                if i >= 2:
                    s_run.wait_event(ev["out"][b])     # step i-2's result has left ybuf[b]
                step(slot=b)
                ev["run"][b].record()
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev["run"][b])
                y_host[b].copy_(ybuf[b], non_blocking=True)
                ev["out"][b].record()
        for st in (s_in, s_run, s_out):
            cur.wait_stream(st)

    e2e_loop(2)
    e2e_steps = max(4, min(args.steps, 20))
    ms_e2e = timed(lambda: e2e_loop(e2e_steps), 1)
    e2e_value = aggregate(T, e2e_steps, ms_e2e, world)
    xbuf[0].copy_(x_host)
    # clocks were sampled from the start of the timed region to here (all of it under load)
    clocks = sampler.stop() if rank == 0 else None

    # ---- the same kernels run dense (k = N_G)
    dense_ms = None
    if not args.no_dense:
        for _ in range(2):
            step(NG)
        run_dense = rotating(lambda c: step(NG, copy=c))
        for _ in range(n_copies):
            run_dense()
        dense_steps = max(3, min(args.steps, 10))
        if flush is None:
            dense_ms = timed(run_dense, dense_steps) / dense_steps
        else:
            dense_ms = 0.0
            for _ in range(dense_steps):
                flush.zero_()
                dense_ms += timed(run_dense, 1) / dense_steps
        step()

    # ---- extra records of the default single-GPU run: seconds-long replay, cuBLAS context, decode sweep
    sustained = cublas = decode_rec = oproj_rec = attn_rec = None
    if world == 1 and not decode and not args.no_extras:
        sustained = sustained_record(torch, run_step, ms_total / args.steps, T, flops_ffn_active(cfg, oproj), peaks, local)
        if not oproj:
            cublas = cublas_dense_context(torch, d)
            if cfg.name == "llama7b_prefill":
                decode_rec = decode_sweep(torch, binding, ctx, peaks, local)
                oproj_rec = oproj_13b_record(torch, binding, ctx, peaks)
                attn_rec = attn_13b_record(torch, binding, ctx, peaks)

    # ---- roofline of the dominant kernel (largest share of the timed region)
    kernels = {n: {"launches": v["launches"], "total_ms": round(v["total_ms"], 4),
                   "share": round(v["total_ms"] / max(sum(p["total_ms"] for p in prof.values()), 1e-9), 4)}
               for n, v in prof.items()}
    dom = max(prof, key=lambda n: prof[n]["total_ms"]) if prof else None
    roofline = None
    if dom:
        avg_s = prof[dom]["total_ms"] / prof[dom]["launches"] * 1e-3
        if decode and dom.startswith("decode_"):
            avg_s = ffn_graph_ms * 1e-3   # the FFN is this one kernel; see ffn_graph_ms above
        tkgd = float(T) * cfg.k * cfg.group * cfg.hidden
        if decode:
            # union of active groups x (gate + up + down) weight bytes, bf16
            union_words = np.bitwise_or.reduce(bits.cpu().numpy().view(np.uint32), axis=0)
            n_union = sum(bin(int(w)).count("1") for w in union_words)
            per_group = cfg.group * cfg.hidden * 2
            bytes_alg = (1.0 if oproj else 3.0) * n_union * per_group   # weights of the groups in the union
            ach = bytes_alg / avg_s / 1e9
            tr, src = ncu_traffic(dom, cfg.name, n_union)
            roofline = roofline_record(dom, "hbm", ach, peaks, tr, src, n_union=n_union)
        else:
            flops_alg = {"prefill_gateup": 4.0 * tkgd, "prefill_down": 2.0 * tkgd, "prefill_down_group": 2.0 * tkgd}.get(dom, 2.0 * tkgd if oproj else 6.0 * tkgd)
            tr, src = ncu_traffic(dom, cfg.name)
            roofline = roofline_record(dom, "tensor", flops_alg / avg_s / 1e12, peaks, tr, src)

    line = None
    if rank == 0:
        ms_step = ms_total / args.steps
        ffn_ms = sum(v["total_ms"] for n, v in prof.items() if n.startswith(("prefill_", "decode_"))) / args.steps
        line = {
            "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_record(cfg, args.op, world, args.flush_l2),
            "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": x_host.numel() * 2,
                    "d2h_bytes_per_step": y_host[0].numel() * 2,
                    "note": "activations cross PCIe every step (pinned host memory, copies of neighbouring "
                            "steps overlap the compute on separate streams); weights are parameters and stay "
                            "resident"},
            "launch": "one CUDA graph replay per step" if not args.no_graph else "direct launches",
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": roofline,
            "kernels": kernels,
            "ffn": {"ms": ffn_ms, "graph_ms": ffn_graph_ms, "active_tflops": flops_ffn_active(cfg, oproj) / (ffn_ms * 1e-3) / 1e12 if ffn_ms else None,
                    "frac_of_bf16_peak": (flops_ffn_active(cfg, oproj) / (ffn_ms * 1e-3) / 1e12 / peaks["bf16_tflops"])
                    if ffn_ms else None},
            "dense": {"ms_per_step": dense_ms, "speedup_vs_dense": (dense_ms / ms_step) if dense_ms else None,
                      "ideal": NG / cfg.k if cfg.k else None},
        }
        if sustained:
            line["sustained"] = sustained
        if cublas:
            cublas["speedup_of_masked_step_over_cublas_dense_ffn"] = cublas["ms"] / ms_step
            line["cublas_dense_context"] = cublas
        if decode_rec:
            line["decode"] = decode_rec
        if oproj_rec:
            line["oproj_13b"] = oproj_rec
        if attn_rec:
            line["attn_13b"] = attn_rec
        if world == 1 and not args.no_cpu_baseline and not oproj:
            sample = min(T, args.oracle_tokens)
            _, ms1 = time_oracle(case, cfg, sample, 1, 0)
            passes = int(min(15, max(1, np.ceil(10e3 / ms1))))     # about 10 s of CPU work in all
            v, ms = time_oracle(case, cfg, sample, passes, 0)
            line["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
                                    "sample": f"first {sample} of {T} tokens, {passes} passes of route, top-k, reorder "
                                              f"and masked FFN in fp64 numpy ({passes * ms / 1e3:.1f} s)"}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()
    return line


# ------------------------------------------------------------------------------- group-sharded FFN
def run_group_sharded(args):
    """--shard groups: tensor parallelism over the pruned dimension.  Every rank holds the gate / up
    rows and the down columns of its contiguous range of groups, routes all tokens (replicated),
    slices the mask to its range, runs reorder + wide_ffn on its shard with an fp32 output, and the
    parts are summed by one NCCL reduce-scatter over the token rows (Eq. 10: the K-axis product is a
    sum over groups).  Total work is fixed as N grows (strong scaling)."""
    import torch
    import torch.distributed as dist

    from paper_2607_28418_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    cfg = make_config(args)
    peaks = load_peaks()
    ctx = binding.Context(local)
    T, NG, G = cfg.tokens, cfg.n_groups, cfg.group
    if T % world:
        raise SystemExit("--shard groups needs tokens divisible by the number of ranks")
    case = synth.make_ffn_case(cfg, 0)                      # the same inputs on every rank
    g0, g1 = binding.group_range(NG, world, rank)
    c0, c1 = g0 * G, g1 * G
    x = binding.upload(case["x"], "bf16")
    w_router = binding.upload(case["w_router"], "bf16")
    wg, wu = binding.upload(case["w_gate"][c0:c1], "bf16"), binding.upload(case["w_up"][c0:c1], "bf16")
    wd = binding.upload(np.ascontiguousarray(case["w_down"][:, c0:c1]), "bf16")
    bits = torch.empty((T, (NG + 31) // 32), dtype=torch.int32, device=dev)
    local_bits = torch.empty((T, max(1, (g1 - g0 + 31) // 32)), dtype=torch.int32, device=dev)
    part = torch.empty((T, cfg.hidden), dtype=torch.float32, device=dev)
    rows = torch.empty((T // world, cfg.hidden), dtype=torch.float32, device=dev)
    y = torch.empty((T // world, cfg.hidden), dtype=torch.bfloat16, device=dev)
    state = {"meta": None}
    shard_ptrs = None
    if args.fused:
        # the fp32 shard of every rank, peer-mapped: the down projection adds into them directly
        if world > 1:
            import torch.distributed._symmetric_memory as symm_mem
            rows = symm_mem.empty((T // world, cfg.hidden), dtype=torch.float32, device=dev)
            handle = symm_mem.rendezvous(rows, dist.group.WORLD)
            shard_ptrs = [int(p) for p in handle.buffer_ptrs]
        else:
            shard_ptrs = [rows.data_ptr()]
        token = torch.zeros((1,), dtype=torch.float32, device=dev)

    def rank_barrier():
        # stream-ordered: a one-element all-reduce on the stream the kernels run on
        if world > 1:
            dist.all_reduce(token)

    def step():
        binding.wide_route(ctx, x, w_router, NG, cfg.k, mask_bits=bits)
        binding.wide_mask_slice(ctx, bits, NG, g0, g1, out=local_bits)
        if T > binding.DECODE_MAX_TOKENS:
            state["meta"] = binding.wide_reorder(ctx, local_bits, g1 - g0, 128, out=state["meta"])
        if args.fused and T > binding.DECODE_MAX_TOKENS:
            rows.zero_()
            rank_barrier()                       # every shard is zero before any rank adds to it
            binding.wide_ffn_tp(ctx, x, wg, wu, wd, G, local_bits, state["meta"], shard_ptrs, T // world)
            rank_barrier()                       # every rank's adds have landed
            y.copy_(rows)
            return
        binding.wide_ffn(ctx, x, wg, wu, wd, G, local_bits, state["meta"], y=part)
        if world > 1:
            dist.reduce_scatter_tensor(rows, part, op=dist.ReduceOp.SUM)
            y.copy_(rows)
        else:
            y.copy_(part)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    if ctx.status() != 0:
        raise RuntimeError("device status word set during warm-up")
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    sync_all()
    ms_total = reduce_max_ms(e0.elapsed_time(e1), world, dev)
    launches = ctx.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    if rank == 0:
        ms_step = ms_total / args.steps
        tfl = flops_ffn_active(cfg) / (ms_step * 1e-3) / 1e12
        rec = config_record(cfg, "ffn", world, args.flush_l2)
        rec["parallelism"] = (f"group-sharded x{world}: each rank holds the weights of a contiguous range of groups, routing "
                              "replicated, " + ("the down projection adds its rows into the owner ranks' fp32 shards over peer "
                                                "memory (reduce-scatter fused into the kernel)" if args.fused else
                                                "fp32 parts summed by one NCCL reduce-scatter over token rows"))
        print(json.dumps({
            "metric": METRIC, "value": T * args.steps / (ms_total * 1e-3), "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": rec,
            "launch": "direct launches", "gpu_launches": int(launches), "clocks": clocks,
            "roofline": roofline_record("whole step (all ranks)", "tensor", tfl, {**peaks, "bf16_tflops": peaks["bf16_tflops"] * world}),
            "note": "the multi-GPU form of this mode has not been run on more than one GPU in this build"}))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------- router forms
def run_route_forms(args):
    """--op route: the three router forms on the workload's shape, each replayed as a graph:
    single linear + top-k, Eq. 4 (bottleneck pair-argmax) with the weight work inside every call, and
    Eq. 4 on the RMSNorm of the hidden state with the weight work prepared once."""
    import torch

    from paper_2607_28418_b200 import binding
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(0)
    cfg = make_config(args)
    ctx = binding.Context(0)
    case = synth.make_ffn_case(cfg, 0)
    pr = synth.make_pair_router(cfg, 0, rank=16)
    x, wr = binding.upload(case["x"], "bf16"), binding.upload(case["w_router"], "bf16")
    w1, w2 = binding.upload(pr["w1"], "bf16"), binding.upload(pr["w2"], "bf16")
    gamma = binding.upload(synth.round_to_bf16((1.0 + 0.1 * np.random.default_rng(1).standard_normal(cfg.hidden)).astype(np.float32)), "bf16")
    NG = cfg.n_groups
    bits = torch.empty((cfg.tokens, (NG + 31) // 32), dtype=torch.int32, device="cuda")
    prepared = binding.wide_route_pair_prepare(ctx, w1, w2, gamma, NG)
    forms = {
        "topk": lambda: binding.wide_route(ctx, x, wr, NG, cfg.k, mask_bits=bits),
        "pair_argmax": lambda: binding.wide_route(ctx, x, w1, NG, mode=binding.ROUTE_PAIR_ARGMAX, w2=w2, rank=16, mask_bits=bits),
        "pair_argmax_rmsnorm_prepared": lambda: binding.wide_route_pair_norm(ctx, x, w1, w2, gamma, 1e-5, prepared, NG, mask_bits=bits),
    }
    out = {}
    for name, fn in forms.items():
        for _ in range(3):
            fn()
        g = graph_of(torch, fn)
        g()
        out[name + "_us"] = round(event_ms(torch, g, max(20, args.steps)) * 1e3, 2)
        ctx.profile_begin(64)
        fn()
        out[name + "_kernels_us"] = {k: round(v["total_ms"] * 1e3, 1) for k, v in ctx.profile_end().items()}
    if ctx.status() != 0:
        raise RuntimeError("device status word set")
    print(json.dumps({"op": "route", "config": config_record(cfg, "route", 1), "rank": 16, **out}))
    ctx.close()


# ------------------------------------------------------------------------------- attention op
def run_attn(args):
    """--op attn: route (attention router) -> reorder -> head-group-masked causal attention on the
    attention half of the workload (one sequence of `tokens` positions, MHA heads of 128)."""
    import torch
    import torch.distributed as dist

    from paper_2607_28418_b200 import binding
    to_dev = binding.upload

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    cfg = make_config(args)
    if not cfg.attn_group:
        raise SystemExit(f"workload {cfg.name} has no attention half")
    peaks = load_peaks()
    ctx = binding.Context(local)
    T, hd = cfg.tokens, 128
    H = cfg.attn_dim // hd
    Hkv = cfg.kv_heads or H                # grouped-query attention when fewer
    hpg = cfg.attn_group // hd
    NG, k = cfg.attn_n_groups, cfg.attn_k
    decode = T <= 8                       # --batch B: B new tokens against a resident K/V cache
    Tk = args.kv_len if args.kv_len else (synth.CONFIGS[args.workload].tokens if decode else T)
    oc = synth.make_oproj_case(cfg, 1000 * rank)
    ac = synth.make_attn_case(1000 * rank, T, Tk, H, Hkv, hd)
    host = {"x": oc["x"], "q": ac["q"].reshape(T, H * hd), "k": ac["k"].reshape(Tk, Hkv * hd), "v": ac["v"].reshape(Tk, Hkv * hd)}
    w_router = to_dev(oc["w_router_attn"], "bf16")
    pinned = {n: torch.from_numpy(synth.to_bf16_bits(a).view(np.int16)).view(torch.bfloat16).pin_memory() for n, a in host.items()}
    bufs = [{n: t.to(dev) for n, t in pinned.items()} for _ in range(2)]
    obuf = [torch.empty((T, H * hd), dtype=torch.bfloat16, device=dev) for _ in range(2)]
    o_host = [torch.empty((T, H * hd), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    bits = torch.empty((T, (NG + 31) // 32), dtype=torch.int32, device=dev)
    state = {"meta": None}

    def attn_only(slot=0):
        b = bufs[slot]
        binding.wide_attn(ctx, b["q"], b["k"], b["v"], H, Hkv, hpg, state["meta"], causal=True, o=obuf[slot],
                          mask_bits=bits if decode else None)

    def step(slot=0, kk=k):
        binding.wide_route(ctx, bufs[slot]["x"], w_router, NG, kk, mask_bits=bits)
        if not decode:
            state["meta"] = binding.wide_reorder(ctx, bits, NG, 128, out=state["meta"])
        attn_only(slot)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sync_all()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        sync_all()
        return reduce_max_ms(e0.elapsed_time(e1), world, dev)

    def graphed(fn):
        if args.no_graph:
            return fn
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g.replay

    for _ in range(max(3, args.warmup)):
        step()
    if ctx.status() != 0:
        raise RuntimeError("device status word set during warm-up")
    run_step = graphed(step)
    run_step()
    sampler = ClockSampler(local)
    sampler.start()
    ms_total = timed(run_step, args.steps)
    value = aggregate(T, args.steps, ms_total, world)
    run_attn_only = graphed(attn_only)
    run_attn_only()
    attn_ms = timed(run_attn_only, args.steps) / args.steps

    launches0 = ctx.launch_count()
    ctx.profile_begin(16 * args.steps + 16)
    for _ in range(args.steps):
        step()
    prof = ctx.profile_end()
    launches = ctx.launch_count() - launches0

    # end to end: x, q, k, v from pinned host memory every step, o back to the host
    s_in, s_run, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev = {n: [torch.cuda.Event(), torch.cuda.Event()] for n in ("in", "run", "out")}

    def e2e_loop(steps):
        cur = torch.cuda.current_stream()
        for st in (s_in, s_run, s_out):
            st.wait_stream(cur)
        for i in range(steps):
            b = i % 2
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev["run"][b])
                for n in pinned:
                    if decode and n in ("k", "v"):
                        continue                        # the K/V cache is resident; only the new tokens travel
                    bufs[b][n].copy_(pinned[n], non_blocking=True)
                ev["in"][b].record()
            with torch.cuda.stream(s_run):
                s_run.wait_event(ev["in"][b])
                if i >= 2:
                    s_run.wait_event(ev["out"][b])
                step(slot=b)
                ev["run"][b].record()
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev["run"][b])
                o_host[b].copy_(obuf[b], non_blocking=True)
                ev["out"][b].record()
        for st in (s_in, s_run, s_out):
            cur.wait_stream(st)

    e2e_loop(2)
    e2e_steps = max(4, min(args.steps, 20))
    ms_e2e = timed(lambda: e2e_loop(e2e_steps), 1)
    clocks = sampler.stop() if rank == 0 else None

    dense_ms = None
    if not args.no_dense:
        for _ in range(2):
            step(kk=NG)
        run_dense = graphed(lambda: step(kk=NG))
        run_dense()
        dense_ms = timed(run_dense, max(3, min(args.steps, 10))) / max(3, min(args.steps, 10))
        step()

    line = None
    if rank == 0:
        # algorithmic FLOPs: every active (token t, head) pair does 4 * d * (t + 1) (QK^T and PV over its keys)
        mask = np.unpackbits(bits.cpu().numpy().view(np.uint8), axis=1, bitorder="little")[:, :NG].astype(bool)
        flops = float((mask.sum(axis=1) * hpg * 4.0 * hd * (np.arange(T) + 1.0 + (Tk - T))).sum())
        ach = flops / (attn_ms * 1e-3) / 1e12
        if decode:
            # algorithmic bytes: K and V rows of every KV head some active query row reads
            heads_read = int(np.repeat(mask.any(axis=0), hpg).reshape(Hkv, H // Hkv).any(axis=1).sum())   # KV heads
            kv_bytes = 2.0 * heads_read * Tk * hd * 2
            roof = roofline_record("attn_decode", "hbm", kv_bytes / (attn_ms * 1e-3) / 1e9, peaks, kv_heads_read=heads_read)
        else:
            tr, src = ncu_traffic("attn_prefill", cfg.name)
            roof = roofline_record("attn_prefill", "tensor", ach, peaks, tr, src)
        kernels = {n: {"launches": v["launches"], "total_ms": round(v["total_ms"], 4),
                       "share": round(v["total_ms"] / max(sum(p["total_ms"] for p in prof.values()), 1e-9), 4)}
                   for n, v in prof.items()}
        line = {
            "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_total / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": cfg.name, "op": "attn", "tokens_per_gpu": T, "keys": Tk, "heads": H, "kv_heads": Hkv, "head_dim": hd,
                       "heads_per_group": hpg, "n_groups": NG, "k": k, "causal": True, "router": cfg.router,
                       "parallelism": f"sequence-sharded x{world} (independent sequences), no collective",
                       "l2": "q, k, v, o of one step are %.0f MB" % ((2 * T * H + 2 * Tk * Hkv) * hd * 2 / 1e6)},
            "e2e": {"value": aggregate(T, e2e_steps, ms_e2e, world), "unit": "tokens/s",
                    "h2d_bytes_per_step": sum(t.numel() * 2 for n, t in pinned.items() if not (decode and n in ("k", "v"))),
                    "d2h_bytes_per_step": o_host[0].numel() * 2},
            "launch": "one CUDA graph replay per step" if not args.no_graph else "direct launches",
            "gpu_launches": int(launches), "clocks": clocks,
            "roofline": roof,
            "kernels": kernels,
            "attn": {"graph_ms": attn_ms, "active_gflop": flops / 1e9},
            "dense": {"ms_per_step": dense_ms, "speedup_vs_dense": (dense_ms / (ms_total / args.steps)) if dense_ms else None,
                      "ideal": NG / k if k else None},
        }
        if world == 1 and not args.no_cpu_baseline:
            sample = min(T, 1024)
            t0 = time.perf_counter()
            m_s = mask[:sample]
            from oracle import wide_oracle as wo
            ks = Tk if decode else sample
            wo.masked_attention(ac["q"][:sample], ac["k"][:ks], ac["v"][:ks], m_s, hpg)
            dt = time.perf_counter() - t0
            line["cpu_baseline"] = {"value": sample / dt, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
                                    "sample": f"first {sample} of {T} positions, masked attention only, fp64 numpy ({dt:.1f} s)"}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b_prefill", choices=sorted(synth.CONFIGS))
    ap.add_argument("--batch", type=int, default=0, help="override the token count (decode batch)")
    ap.add_argument("--router", default="", choices=["", "random", "clustered", "clustered_corr"])
    ap.add_argument("--k", type=int, default=None)
    ap.add_argument("--group", type=int, default=0)
    ap.add_argument("--op", default="ffn", choices=["ffn", "oproj", "attn", "qproj", "route"],
                    help="oproj, qproj and attn need a workload with an attention half")
    ap.add_argument("--shard", default="tokens", choices=["tokens", "groups"],
                    help="multi-GPU partition: token shards with replicated weights (no collective), or group "
                         "shards (tensor parallel over the pruned dimension) with one reduce-scatter per step")
    ap.add_argument("--fused", action="store_true",
                    help="--shard groups: fuse the reduce-scatter into the down projection (adds over peer memory)")
    ap.add_argument("--premasked", action="store_true",
                    help="oproj: feed an attention output that already has zeros for inactive pairs")
    ap.add_argument("--kaxis", default="auto", choices=["auto", "group", "owner"],
                    help="prefill K-axis kernel (down / output projection): per-group scatter-reduce, owner-computes, "
                         "or the library's own choice")
    ap.add_argument("--decode-tc", action="store_true",
                    help="decode with one or two tokens: the tensor-core kernel instead of the matrix-vector kernel")
    ap.add_argument("--reduce-bf16", action="store_true", help="per-group K-axis kernel: add partial sums in bf16")
    ap.add_argument("--kv-len", type=int, default=0, help="attn: number of keys (default: the workload's tokens)")
    ap.add_argument("--flush-l2", action="store_true")
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel directly instead of replaying a graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the seconds-long replay, the cuBLAS context row and the decode batch sweep")
    ap.add_argument("--oracle-tokens", type=int, default=4096, help="tokens of the workload the CPU oracle runs")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.op == "route":
        run_route_forms(args)
    elif args.shard == "groups":
        run_group_sharded(args)
    elif args.op == "attn":
        run_attn(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
