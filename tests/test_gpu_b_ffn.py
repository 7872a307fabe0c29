"""GPU parity: wide_ffn / wide_oproj (CUDA-core, tcgen05 prefill and decode paths) vs the oracle.

Stage-wise: each stage gets the oracle's mask / metadata as input, so a routing difference
cannot hide as an FFN error.  Float bar: max|err| <= 2e-2 * max|ref|.
"""
import numpy as np
import pytest
import torch

from oracle import wide_oracle as wo
from paper_2607_28418_b200 import synth
from tests.gpu_util import assert_close, bits_to_dev, meta_to_dev, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_28418_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


def _ffn_inputs(cfg, seed, mask=None):
    case = synth.make_ffn_case(cfg, seed)
    if mask is None:
        mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router"]), cfg.k)
    dev = {k: to_dev(case[k], cfg.dtype) for k in ("x", "w_gate", "w_up", "w_down")}
    return case, mask, dev


def _run_ffn(ctx, cfg, seed, flags, mask=None, out_dtype=None, with_meta=True, clustered_order=True):
    from paper_2607_28418_b200 import binding
    case, mask, dev = _ffn_inputs(cfg, seed, mask)
    ref = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"], mask, cfg.group)
    bits = bits_to_dev(wo.pack_mask_bits(mask))
    meta = meta_to_dev(wo.reorder(mask, 128)) if with_meta else None
    if meta is not None and not clustered_order:
        meta.pop("token_order")
        meta.pop("token_rank")
    y = binding.wide_ffn(ctx, dev["x"], dev["w_gate"], dev["w_up"], dev["w_down"], cfg.group, bits, meta,
                         out_dtype=out_dtype, flags=flags)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    return y, ref, mask


# ----------------------------------------------------------------------------- CUDA-core path
def test_tiny_config_fp32_simt(ctx):
    from paper_2607_28418_b200 import binding
    cfg = synth.CONFIGS["tiny"]
    y, ref, _ = _run_ffn(ctx, cfg, 0, binding.FLAG_SIMT, with_meta=False)
    assert_close(y, ref, "tiny fp32", rel=1e-4)


@pytest.mark.parametrize("T,D,Dff,G,k,dtype", [(70, 96, 320, 32, 5, "fp32"), (130, 128, 512, 16, 9, "bf16"),
                                               (33, 64, 256, 64, 0, "bf16"), (33, 64, 256, 64, 4, "bf16")])
def test_simt_odd_shapes(ctx, T, D, Dff, G, k, dtype):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=T, hidden=D, d_ff=Dff, group=G, k=k, dtype=dtype)
    y, ref, _ = _run_ffn(ctx, cfg, 1, binding.FLAG_SIMT, with_meta=False)
    if k == 0:
        assert (y.float().cpu().numpy() == 0).all()
    else:
        assert_close(y, ref, f"simt {T}x{D}x{Dff}")


# ----------------------------------------------------------------------------- tcgen05 prefill
@pytest.mark.parametrize("T,D,Dff,G,k", [(128, 256, 512, 128, 2), (300, 512, 1024, 128, 4),
                                         (257, 512, 1024, 64, 8), (200, 256, 1024, 256, 2),
                                         (640, 1024, 2048, 128, 8)])
def test_prefill_tc_matches_oracle(ctx, T, D, Dff, G, k):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=T, hidden=D, d_ff=Dff, group=G, k=k)
    y, ref, _ = _run_ffn(ctx, cfg, 2, binding.FLAG_FORCE_PREFILL)
    assert_close(y, ref, f"prefill tc {T}x{D}x{Dff} G{G}")


@pytest.mark.parametrize("T,D,Dff,G,k,out", [(1280, 4096, 256, 128, 1, None), (1100, 4096, 512, 64, 5, torch.float32)])
def test_prefill_tc_more_tiles_than_sms(ctx, T, D, Dff, G, k, out):
    """More output tiles than SMs with a ragged remainder (both tile heights of the down
    projection get exercised across the parametrisations); run twice: same result."""
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=T, hidden=D, d_ff=Dff, group=G, k=k)
    y1, ref, _ = _run_ffn(ctx, cfg, 8, binding.FLAG_FORCE_PREFILL, out_dtype=out)
    assert_close(y1, ref, f"many tiles {T}x{D}x{Dff}")
    y2, _, _ = _run_ffn(ctx, cfg, 8, binding.FLAG_FORCE_PREFILL, out_dtype=out)
    assert_close(y2, ref, f"many tiles, second call {T}x{D}x{Dff}")


def test_prefill_tc_fp32_output_and_variable_budget(ctx):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=384, hidden=512, d_ff=1024, group=128, k=4)
    ctx.workspace(1 << 20).fill_(0xFF)              # stale scratch (NaN patterns) must not leak into y
    mask = synth.bernoulli_mask(3, 384, 8, 0.4)     # variable active groups per token
    mask[5] = False                                  # a token with nothing active -> zero row
    mask[:, 6] = False                               # a group nobody selects -> skipped block column
    y, ref, _ = _run_ffn(ctx, cfg, 3, binding.FLAG_FORCE_PREFILL, mask=mask, out_dtype=torch.float32)
    assert_close(y, ref, "prefill tc fp32 out")
    assert (y[5] == 0).all()


def test_prefill_tc_closed_cases(ctx):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=256, hidden=256, d_ff=512, group=128, k=4)
    ones = np.ones((256, 4), dtype=bool)
    y, ref, _ = _run_ffn(ctx, cfg, 4, binding.FLAG_FORCE_PREFILL, mask=ones)        # dense SwiGLU
    assert_close(y, ref, "all-ones")
    y, _, _ = _run_ffn(ctx, cfg, 4, binding.FLAG_FORCE_PREFILL, mask=~ones)         # exact zero
    assert (y.float().cpu().numpy() == 0).all()
    # clustered: first half of the tokens uses groups {0,1}, second half {2,3}: whole blocks skipped
    m = np.zeros((256, 4), dtype=bool)
    m[:128, :2] = True
    m[128:, 2:] = True
    y, ref, _ = _run_ffn(ctx, cfg, 4, binding.FLAG_FORCE_PREFILL, mask=m)
    assert_close(y, ref, "block-clustered")


def test_prefill_tc_token_order_is_optional_and_does_not_change_the_result(ctx):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=700, hidden=512, d_ff=2048, group=128, k=6, router="clustered")
    y1, ref, mask = _run_ffn(ctx, cfg, 14, binding.FLAG_FORCE_PREFILL)
    y2, _, _ = _run_ffn(ctx, cfg, 14, binding.FLAG_FORCE_PREFILL, clustered_order=False)
    assert len({r.tobytes() for r in mask}) <= 4
    assert_close(y1, ref, "clustered order")
    assert_close(y2, ref, "original order")
    assert_close(y1, y2.float().cpu().numpy().astype(np.float64), "same result either way", rel=1e-2)


def test_prefill_tc_token_level_skipping_is_the_one_decision_per_token_case(ctx):
    """M-axis (dynamic depth) routing of Section 3.3: one decision per token for the whole FFN is
    the mask whose columns are all equal; skipped tokens give exact zeros."""
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("depth", tokens=700, hidden=512, d_ff=1024, group=128, k=8)
    rng = np.random.default_rng(21)
    keep = rng.random(cfg.tokens) < 0.4
    mask = np.repeat(keep[:, None], cfg.n_groups, axis=1)
    y, ref, _ = _run_ffn(ctx, cfg, 6, binding.FLAG_FORCE_PREFILL, mask=mask)
    assert (y.float().cpu().numpy()[~keep] == 0.0).all()
    assert_close(y, ref, "token-level skipping")


def test_prefill_tc_agrees_with_simt_and_is_deterministic(ctx):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=300, hidden=512, d_ff=1024, group=128, k=4)
    y1, ref, mask = _run_ffn(ctx, cfg, 6, binding.FLAG_FORCE_PREFILL)
    y2, _, _ = _run_ffn(ctx, cfg, 6, binding.FLAG_FORCE_PREFILL)
    assert torch.equal(y1, y2)
    y3, _, _ = _run_ffn(ctx, cfg, 6, binding.FLAG_SIMT, with_meta=False)
    assert_close(y1, y3.float().cpu().numpy().astype(np.float64), "tc vs simt")


# ----------------------------------------------------------------------------- decode
@pytest.mark.parametrize("B", [1, 8, 33, 64])
@pytest.mark.parametrize("G", [64, 128, 256])
def test_decode_matches_oracle(ctx, B, G):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=B, hidden=512, d_ff=2048, group=G, k=2048 // G // 2)
    y, ref, _ = _run_ffn(ctx, cfg, 7 + B, binding.FLAG_NONE, with_meta=False)
    assert_close(y, ref, f"decode B{B} G{G}")


@pytest.mark.parametrize("B", [2, 3, 4])
def test_decode_tiny_batches(ctx, B):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=B, hidden=1024, d_ff=2048, group=128, k=7)
    y, ref, _ = _run_ffn(ctx, cfg, 20 + B, binding.FLAG_NONE, with_meta=False, out_dtype=torch.float32)
    assert_close(y, ref, f"decode B{B}")


def test_decode_clustered_union_and_zero_cases(ctx):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=16, hidden=512, d_ff=2048, group=128, k=8, router="clustered")
    y, ref, mask = _run_ffn(ctx, cfg, 11, binding.FLAG_NONE, with_meta=False)
    assert len({r.tobytes() for r in mask}) <= 4
    assert_close(y, ref, "decode clustered")
    zero = np.zeros((16, 16), dtype=bool)
    y, _, _ = _run_ffn(ctx, cfg, 11, binding.FLAG_NONE, mask=zero, with_meta=False)
    assert (y.float().cpu().numpy() == 0).all()
    y1, ref, _ = _run_ffn(ctx, cfg, 11, binding.FLAG_NONE, mask=~zero, with_meta=False, out_dtype=torch.float32)
    assert_close(y1, ref, "decode dense fp32 out")


def test_decode_calls_of_different_shapes_share_one_context(ctx):
    """The decode kernels keep fp32 sums, counters and a barrier in buffers owned by the context
    (cleared by the kernels themselves, not by the host).  A sequence of calls whose shapes place
    those sums differently -- small then large batch, narrow then wide layer, FFN then O-projection
    and back -- must leave every call with clean sums."""
    from paper_2607_28418_b200 import binding
    seq = [("ffn", 5, 512, 2048, 128), ("ffn", 64, 1024, 4096, 128), ("oproj", 32, 512, 1024, 512),
           ("ffn", 3, 1024, 2048, 64), ("oproj", 1, 1024, 512, 256), ("ffn", 64, 512, 2048, 256),
           ("ffn", 16, 1024, 4096, 128)]
    for i, (kind, B, D, inner, G) in enumerate(seq):
        if kind == "ffn":
            cfg = synth.WideConfig("t", tokens=B, hidden=D, d_ff=inner, group=G, k=max(1, inner // G // 2))
            y, ref, _ = _run_ffn(ctx, cfg, 40 + i, binding.FLAG_NONE, with_meta=False)
        else:
            y, ref = _run_oproj(ctx, B, D, inner, G, 1, binding.FLAG_NONE, seed=40 + i)
        assert_close(y, ref, f"call {i}: {kind} B{B} D{D} inner{inner} G{G}")


# ----------------------------------------------------------------------------- O-projection
def _run_oproj(ctx, T, D, K, G, k, flags, dtype="bf16", seed=0):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=T, hidden=D, d_ff=D, group=64, k=1, dtype=dtype, attn_dim=K, attn_group=G,
                           attn_k=k)
    case = synth.make_oproj_case(cfg, seed)
    mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router_attn"]), k)
    ref = wo.oproj(case["attn_out"], case["w_o"], mask, G)
    y = binding.wide_oproj(ctx, to_dev(case["attn_out"], dtype), to_dev(case["w_o"], dtype), G,
                           bits_to_dev(wo.pack_mask_bits(mask)), meta_to_dev(wo.reorder(mask, 128)), flags=flags)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    return y, ref


def test_oproj_simt_fp32(ctx):
    from paper_2607_28418_b200 import binding
    y, ref = _run_oproj(ctx, 100, 96, 160, 32, 2, binding.FLAG_SIMT, dtype="fp32")
    assert_close(y, ref, "oproj simt fp32", rel=1e-4)


@pytest.mark.parametrize("T,D,K,G,k", [(300, 512, 1024, 512, 1), (256, 256, 1024, 128, 3), (130, 512, 512, 64, 4)])
def test_oproj_prefill_tc(ctx, T, D, K, G, k):
    from paper_2607_28418_b200 import binding
    y, ref = _run_oproj(ctx, T, D, K, G, k, binding.FLAG_FORCE_PREFILL)
    assert_close(y, ref, f"oproj prefill {T}x{D}x{K} G{G}")


def test_oproj_prefill_with_an_input_that_is_already_masked(ctx):
    """The output of wide_attn has zeros for inactive pairs; the O-projection then needs no masking pass."""
    from paper_2607_28418_b200 import binding
    T, D, K, G, k = 700, 512, 1024, 128, 3
    rng = np.random.default_rng(8)
    a = synth.make_activations(rng, T, K, "bf16", "random")
    w_o = synth.make_weight(rng, D, K, 0.02, "bf16")
    mask = synth.random_mask(9, T, K // G, k)
    a_masked = (a * wo.expand_group_mask(mask, G)).astype(np.float32)
    y = binding.wide_oproj(ctx, to_dev(a_masked, "bf16"), to_dev(w_o, "bf16"), G, bits_to_dev(wo.pack_mask_bits(mask)),
                           meta_to_dev(wo.reorder(mask, 128)), flags=binding.FLAG_INPUT_MASKED)
    assert_close(y, wo.oproj(a, w_o, mask, G), "oproj, masked input")


@pytest.mark.parametrize("B", [1, 32])
def test_oproj_decode(ctx, B):
    from paper_2607_28418_b200 import binding
    y, ref = _run_oproj(ctx, B, 512, 1024, 512, 1, binding.FLAG_NONE)
    assert_close(y, ref, f"oproj decode B{B}")
