"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.

Integer stages (mask, permutation, tile map) are compared in full and bit-exact.  Float outputs
are compared element by element over EVERY token row and every attention head: the oracle computes
the rows a block at a time (an output row depends only on its own token and mask row, Eq. 3 /
Eq. 2; attention heads are independent, Eq. 1).
"""
import numpy as np
import pytest
import torch

from oracle import wide_oracle as wo
from paper_2607_28418_b200 import synth
from tests.gpu_util import REL_TOL, assert_all_rows_close, bits_to_dev, bits_to_host, ffn_ref_rows, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_28418_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


def _chain(ctx, cfg, seed):
    from paper_2607_28418_b200 import binding
    case = synth.make_ffn_case(cfg, seed)
    d = {k: to_dev(v, cfg.dtype) for k, v in case.items()}
    NG, T = cfg.n_groups, cfg.tokens
    bits, _ = binding.wide_route(ctx, d["x"], d["w_router"], NG, cfg.k)
    mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router"]), cfg.k)
    assert (bits_to_host(bits) == wo.pack_mask_bits(mask)).all(), "mask bits differ"
    meta = None
    if T > 64:
        meta = binding.wide_reorder(ctx, bits, NG, 128)
        ref = wo.reorder(mask, 128)
        assert (meta["perm"].cpu().numpy() == ref["perm"]).all()
        assert (meta["counts"].cpu().numpy() == ref["counts"]).all()
        assert (meta["tile_map"].cpu().numpy() == ref["tile_map"]).all()
        nw = int(meta["n_work"].item())
        assert nw == ref["n_work"] and (meta["work_list"].cpu().numpy()[:nw] == ref["work_list"]).all()
        assert (meta["offsets"].cpu().numpy() == ref["offsets"]).all()
    y = binding.wide_ffn(ctx, d["x"], d["w_gate"], d["w_up"], d["w_down"], cfg.group, bits, meta)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    return assert_all_rows_close(y, ffn_ref_rows(case, mask, cfg.group), cfg.name)


def test_llama7b_prefill_chain(ctx):
    rel = _chain(ctx, synth.CONFIGS["llama7b_prefill"], 0)
    print("llama7b_prefill rel err", rel)


@pytest.mark.parametrize("B,seed", [(1, 0), (8, 1), (32, 2), (64, 3)])
def test_llama8b_decode_chain(ctx, B, seed):
    cfg = synth.CONFIGS["llama8b_decode"].with_(tokens=B, router="clustered" if seed % 2 else "random")
    _chain(ctx, cfg, seed)


def test_llama13b_layer_oproj_and_ffn(ctx):
    from paper_2607_28418_b200 import binding
    cfg = synth.CONFIGS["llama13b_layer"]
    case = synth.make_oproj_case(cfg, 0)
    NG, G, T = cfg.attn_n_groups, cfg.attn_group, cfg.tokens
    d = {k: to_dev(v, cfg.dtype) for k, v in case.items()}
    bits, _ = binding.wide_route(ctx, d["x"], d["w_router_attn"], NG, cfg.attn_k)
    mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router_attn"]), cfg.attn_k)
    assert (bits_to_host(bits) == wo.pack_mask_bits(mask)).all()
    meta = binding.wide_reorder(ctx, bits, NG, 128)
    assert (meta["perm"].cpu().numpy() == wo.reorder(mask, 128)["perm"]).all()
    y = binding.wide_oproj(ctx, d["attn_out"], d["w_o"], G, bits, meta)
    assert_all_rows_close(y, wo.oproj(case["attn_out"], case["w_o"], mask, G), "13B O-projection, every row")
    # decode batch 32 of the same layer
    y32 = binding.wide_oproj(ctx, d["attn_out"][:32].contiguous(), d["w_o"], G, bits[:32].contiguous(), None)
    y_ref = wo.oproj(case["attn_out"][:32], case["w_o"], mask[:32], G)
    assert np.abs(y32.float().cpu().numpy() - y_ref).max() <= REL_TOL * np.abs(y_ref).max()
    assert ctx.status() == 0
    # FFN half of the layer, prefill
    _chain(ctx, cfg, 1)


def test_llama13b_layer_attention_and_qproj(ctx):
    """Masked attention and the routed Q projection at the 13B layer's full size (one causal
    sequence of 4096 positions, 40 heads of 128, 10 routing groups).  Attention heads are
    independent and every one of them is compared; so is every row of the Q projection."""
    from paper_2607_28418_b200 import binding
    cfg = synth.CONFIGS["llama13b_layer"]
    T, hd = cfg.tokens, 128
    H, hpg, NG = cfg.attn_dim // hd, cfg.attn_group // hd, cfg.attn_n_groups
    case = synth.make_oproj_case(cfg, 0)
    xd, wr = to_dev(case["x"], "bf16"), to_dev(case["w_router_attn"], "bf16")
    bits, _ = binding.wide_route(ctx, xd, wr, NG, cfg.attn_k)
    mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router_attn"]), cfg.attn_k)
    assert (bits_to_host(bits) == wo.pack_mask_bits(mask)).all()
    meta = binding.wide_reorder(ctx, bits, NG, 128)
    ac = synth.make_attn_case(0, T, T, H, H, hd)
    o = binding.wide_attn(ctx, to_dev(ac["q"].reshape(T, -1), "bf16"), to_dev(ac["k"].reshape(T, -1), "bf16"),
                          to_dev(ac["v"].reshape(T, -1), "bf16"), H, H, hpg, meta)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    got = o.float().cpu().numpy().reshape(T, H, hd)
    head_mask = np.repeat(mask, hpg, axis=1)
    assert (got[~head_mask] == 0.0).all()
    for h in range(H):
        g = h // hpg
        ref = wo.masked_attention(ac["q"][:, h:h + 1], ac["k"][:, h:h + 1], ac["v"][:, h:h + 1], mask[:, g:g + 1], 1)
        err = np.abs(got[:, h] - ref[:, 0]).max()
        assert err <= REL_TOL * np.abs(ref).max(), f"head {h}: {err:.3e}"
    # routed Q projection, every row
    wq = synth.make_weight(np.random.default_rng(3), cfg.attn_dim, cfg.hidden, 0.02, "bf16")
    yq = binding.wide_qproj(ctx, xd, to_dev(wq, "bf16"), cfg.attn_group, meta)
    ref = wo.qproj(case["x"], wq, mask, cfg.attn_group)
    assert (yq.float().cpu().numpy()[~wo.expand_group_mask(mask, cfg.attn_group)] == 0.0).all()
    assert_all_rows_close(yq, ref, "13B routed Q projection, every row")
    assert ctx.status() == 0


def test_llama8b_layer_grouped_query_attention(ctx):
    """Grouped-query attention at the 8B layer's full size: 32 query heads on 8 KV heads of 128, one
    causal sequence of 4096 positions, 8 routing groups of 4 query heads, 4 active per token.  Prefill
    form and decode form (one new token against the same 4096 keys), every head compared."""
    from paper_2607_28418_b200 import binding
    cfg = synth.CONFIGS["llama8b_layer"]
    T, hd = cfg.tokens, 128
    H, Hkv, hpg, NG = cfg.attn_dim // hd, cfg.kv_heads, cfg.attn_group // hd, cfg.attn_n_groups
    rep = H // Hkv
    case = synth.make_oproj_case(cfg, 0)
    mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router_attn"]), cfg.attn_k)
    bits = bits_to_dev(wo.pack_mask_bits(mask))
    meta = binding.wide_reorder(ctx, bits, NG, 128)
    ac = synth.make_attn_case(0, T, T, H, Hkv, hd)
    qd, kd, vd = to_dev(ac["q"].reshape(T, -1), "bf16"), to_dev(ac["k"].reshape(T, -1), "bf16"), to_dev(ac["v"].reshape(T, -1), "bf16")
    o = binding.wide_attn(ctx, qd, kd, vd, H, Hkv, hpg, meta)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    got = o.float().cpu().numpy().reshape(T, H, hd)
    head_mask = np.repeat(mask, hpg, axis=1)
    assert (got[~head_mask] == 0.0).all()
    for h in range(H):
        g, kv = h // hpg, h // rep
        ref = wo.masked_attention(ac["q"][:, h:h + 1], ac["k"][:, kv:kv + 1], ac["v"][:, kv:kv + 1], mask[:, g:g + 1], 1)
        err = np.abs(got[:, h] - ref[:, 0]).max()
        assert err <= REL_TOL * np.abs(ref).max(), f"head {h}: {err:.3e}"
    # decode form: the last position as a new token against the whole cache
    q1 = to_dev(ac["q"][T - 1:T].reshape(1, -1), "bf16")
    m1 = mask[T - 1:T]
    o1 = binding.wide_attn(ctx, q1, kd, vd, H, Hkv, hpg, None, causal=True, mask_bits=bits_to_dev(wo.pack_mask_bits(m1)))
    torch.cuda.synchronize()
    assert ctx.status() == 0
    ref1 = wo.masked_attention(ac["q"][T - 1:T], ac["k"], ac["v"], m1, hpg)
    g1 = o1.float().cpu().numpy().reshape(1, H, hd)
    assert (g1[~np.repeat(m1, hpg, axis=1)] == 0.0).all()
    assert np.abs(g1 - ref1).max() <= REL_TOL * np.abs(ref1).max()
    # and it is what the prefill form gave for that position
    assert np.abs(g1[0] - got[T - 1]).max() <= REL_TOL * np.abs(ref1).max()


def test_llama13b_layer_attention_decode_long_cache(ctx):
    """The decode form at the size the benchmark times: one new token against a cache of 32 768
    keys, 40 heads of 128, five of ten head groups active (both kernels: TMA ring and plain loads).
    Every head is checked: the oracle's cost is one row of scores per head."""
    from paper_2607_28418_b200 import binding
    cfg = synth.CONFIGS["llama13b_layer"]
    hd, Tk = 128, 32768
    H, hpg, NG = cfg.attn_dim // hd, cfg.attn_group // hd, cfg.attn_n_groups
    ac = synth.make_attn_case(4, 1, Tk, H, H, hd)
    mask = synth.random_mask(9, 1, NG, cfg.attn_k)
    bits = bits_to_dev(wo.pack_mask_bits(mask))
    qd, kd, vd = (to_dev(ac[n].reshape(-1, H * hd), "bf16") for n in ("q", "k", "v"))
    ref = wo.masked_attention(ac["q"], ac["k"], ac["v"], mask, hpg)
    head_mask = np.repeat(mask, hpg, axis=1)
    for flags in (0, binding.FLAG_SIMT):
        o = binding.wide_attn(ctx, qd, kd, vd, H, H, hpg, None, causal=True, mask_bits=bits, flags=flags)
        torch.cuda.synchronize()
        assert ctx.status() == 0
        got = o.float().cpu().numpy().reshape(1, H, hd)
        assert (got[~head_mask] == 0.0).all()
        assert np.abs(got - ref).max() <= REL_TOL * np.abs(ref).max()


def test_prefill_four_times_the_largest_config(ctx):
    """T = 16384 on the 8B shape: index arithmetic past the configs' sizes (perm of 1.8 M entries,
    H of 235 M elements), several waves of tiles in every kernel."""
    _chain(ctx, synth.CONFIGS["llama8b_prefill"].with_(tokens=16384), 3)
