"""GPU parity of group sharding (tensor parallelism over the pruned dimension, Eq. 10 as a sum over
group ranges): every rank's part, computed by the ordinary entry points on that rank's weight shard
with the sliced mask, against the oracle's result for that group range alone, and the sum of the
parts against the oracle's full result.  The ranks are emulated one after the other on one GPU (no
rank waits on another: the parts are independent until the final sum)."""
import numpy as np
import pytest
import torch

from oracle import wide_oracle as wo
from paper_2607_28418_b200 import synth
from tests.gpu_util import REL_TOL, assert_close, bits_to_dev, bits_to_host, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_28418_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


@pytest.mark.parametrize("NG,ranges", [(86, [(0, 22), (22, 43), (43, 65), (65, 86)]), (224, [(28 * r, 28 * r + 28) for r in range(8)]),
                                       (70, [(31, 33), (0, 70), (5, 5), (63, 65), (32, 64)]), (10, [(0, 5), (5, 10)])])
def test_mask_slice_bit_exact(ctx, NG, ranges):
    from paper_2607_28418_b200 import binding
    mask = synth.bernoulli_mask(NG, 333, NG, 0.5)
    bits = bits_to_dev(wo.pack_mask_bits(mask))
    for g0, g1 in ranges:
        out = binding.wide_mask_slice(ctx, bits, NG, g0, g1)
        if g1 > g0:
            assert (bits_to_host(out) == wo.pack_mask_bits(mask[:, g0:g1])).all(), (g0, g1)
    with pytest.raises(binding.WideError):
        binding.wide_mask_slice(ctx, bits, NG, 3, NG + 1)


def _ffn_parts(ctx, cfg, seed, world, flags=0):
    from paper_2607_28418_b200 import binding
    case = synth.make_ffn_case(cfg, seed)
    NG, G, T = cfg.n_groups, cfg.group, cfg.tokens
    mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router"]), cfg.k)
    bits = bits_to_dev(wo.pack_mask_bits(mask))
    xd = to_dev(case["x"], "bf16")
    full_ref = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"], mask, G)
    total = torch.zeros((T, cfg.hidden), dtype=torch.float32, device="cuda")
    for r in range(world):
        g0, g1 = binding.group_range(NG, world, r)
        c0, c1 = g0 * G, g1 * G
        wg, wu = to_dev(case["w_gate"][c0:c1], "bf16"), to_dev(case["w_up"][c0:c1], "bf16")
        wd = to_dev(np.ascontiguousarray(case["w_down"][:, c0:c1]), "bf16")          # this rank's shard, contiguous
        local_bits = binding.wide_mask_slice(ctx, bits, NG, g0, g1)
        meta = binding.wide_reorder(ctx, local_bits, g1 - g0, 128) if T > 64 else None
        part = binding.wide_ffn(ctx, xd, wg, wu, wd, G, local_bits, meta, out_dtype=torch.float32, flags=flags)
        torch.cuda.synchronize()
        assert ctx.status() == 0
        only = np.zeros_like(mask)
        only[:, g0:g1] = mask[:, g0:g1]
        part_ref = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"], only, G)
        err = np.abs(part.cpu().numpy().astype(np.float64) - part_ref).max()
        assert err <= REL_TOL * np.abs(full_ref).max(), f"rank {r} of {world}: {err:.3e}"
        total += part
    assert_close(total, full_ref, f"sum of {world} parts")


@pytest.mark.parametrize("world", [2, 4, 8])
def test_ffn_prefill_parts_add_up(ctx, world):
    _ffn_parts(ctx, synth.WideConfig("tp", tokens=640, hidden=512, d_ff=4096, group=128, k=12), 3, world)


def test_ffn_prefill_parts_add_up_uneven_ranges(ctx):
    # 22 groups over 4 ranks: 6, 6, 5, 5
    _ffn_parts(ctx, synth.WideConfig("tp", tokens=300, hidden=512, d_ff=22 * 64, group=64, k=9), 4, 4)


@pytest.mark.parametrize("world", [2, 4])
def test_ffn_decode_parts_add_up(ctx, world):
    _ffn_parts(ctx, synth.WideConfig("tp", tokens=16, hidden=512, d_ff=2048, group=128, k=8), 5, world)


@pytest.mark.parametrize("world,flags", [(2, 0), (4, 0), (2, 16)])
def test_oproj_parts_add_up(ctx, world, flags):
    from paper_2607_28418_b200 import binding
    T, D, K, G, k = 700, 512, 2048, 256, 3
    NG = K // G
    rng = np.random.default_rng(12)
    a = synth.make_activations(rng, T, K, "bf16", "random")
    w_o = synth.make_weight(rng, D, K, 0.02, "bf16")
    mask = synth.random_mask(13, T, NG, k)
    bits = bits_to_dev(wo.pack_mask_bits(mask))
    total = torch.zeros((T, D), dtype=torch.float32, device="cuda")
    for r in range(world):
        g0, g1 = binding.group_range(NG, world, r)
        local_bits = binding.wide_mask_slice(ctx, bits, NG, g0, g1)
        meta = binding.wide_reorder(ctx, local_bits, g1 - g0, 128)
        a_r = to_dev(np.ascontiguousarray(a[:, g0 * G:g1 * G]), "bf16")
        w_r = to_dev(np.ascontiguousarray(w_o[:, g0 * G:g1 * G]), "bf16")
        total += binding.wide_oproj(ctx, a_r, w_r, G, local_bits, meta, out_dtype=torch.float32,
                                    flags=binding.FLAG_FORCE_PREFILL | flags)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    assert_close(total, wo.oproj(a, w_o, mask, G), f"O-projection, sum of {world} parts")


@pytest.mark.parametrize("T,world", [(640, 2), (640, 4), (1100, 8), (2048, 4)])
def test_fused_reduce_scatter_adds_every_part_into_the_owners_shard(ctx, T, world):
    """wide_ffn_tp: the down projection's epilogue adds this rank's part of every token row into the
    fp32 shard of the rank that owns the row.  The ranks are emulated one after the other on one GPU
    (the adds are one-sided: no rank waits on another); their shards are separate local buffers, the
    same instruction that would cross NVLink adds into them.  Shards concatenated = the full FFN."""
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("tp", tokens=T, hidden=512, d_ff=4096, group=128, k=12, router="clustered" if world == 8 else "random")
    case = synth.make_ffn_case(cfg, 7)
    NG, G = cfg.n_groups, cfg.group
    mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router"]), cfg.k)
    bits = bits_to_dev(wo.pack_mask_bits(mask))
    xd = to_dev(case["x"], "bf16")
    rows_per_rank = (T + world - 1) // world
    shards = [torch.zeros((rows_per_rank, cfg.hidden), dtype=torch.float32, device="cuda") for _ in range(world)]
    ptrs = [t.data_ptr() for t in shards]
    for r in range(world):
        g0, g1 = binding.group_range(NG, world, r)
        c0, c1 = g0 * G, g1 * G
        wg, wu = to_dev(case["w_gate"][c0:c1], "bf16"), to_dev(case["w_up"][c0:c1], "bf16")
        wd = to_dev(np.ascontiguousarray(case["w_down"][:, c0:c1]), "bf16")
        local_bits = binding.wide_mask_slice(ctx, bits, NG, g0, g1)
        meta = binding.wide_reorder(ctx, local_bits, g1 - g0, 128)
        binding.wide_ffn_tp(ctx, xd, wg, wu, wd, G, local_bits, meta, ptrs, rows_per_rank)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    y = torch.cat(shards, dim=0)[:T]
    ref = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"], mask, G)
    assert_close(y, ref, f"fused reduce-scatter, {world} ranks")
    if world * rows_per_rank > T:
        assert (torch.cat(shards, dim=0)[T:] == 0).all().item()     # rows past the batch are never touched
