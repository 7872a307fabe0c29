"""wide_route_static: routing for hosts that must not allocate device memory.

A serving process that gave its whole device heap to its own pool, or a plugin that runs while
another framework holds its allocator lock, cannot hand wide_route a workspace.  The static
variant keeps its fp64 score scratch in a fixed array inside the library instead.  This test
calls it through the C ABI twice in a row, with different inputs, and checks each result against
the ordinary entry point (the masks bit for bit, the scores within float32 round-off) and against
the CPU oracle's fp64 decision (bit for bit).  It also
checks that a problem larger than the fixed array is refused.  The file sorts last so that a run
that stops at the first failure has already exercised everything else.
"""
import numpy as np
import pytest
import torch

from oracle import wide_oracle as wo
from paper_2607_28418_b200 import synth
from tests.gpu_util import bits_to_host, to_dev

pytestmark = pytest.mark.gpu


def _case(seed, T, D, NG):
    cfg = synth.WideConfig("t", tokens=T, hidden=D, d_ff=NG * 64, group=64, k=NG // 2)
    c = synth.make_ffn_case(cfg, seed)
    return to_dev(c["x"], "bf16"), to_dev(c["w_router"], "bf16"), c


def test_static_route_matches_workspace_route_twice_in_a_row():
    from paper_2607_28418_b200 import binding
    ctx = binding.Context(0)
    try:
        # second call is smaller than the first, so stale scratch from call one lies beyond and
        # inside the region call two uses
        for seed, (T, D, NG, k) in enumerate([(480, 1024, 112, 56), (300, 512, 86, 43)]):
            x, wr, host = _case(seed, T, D, NG)
            ref_bits, ref_scores = binding.wide_route(ctx, x, wr, NG, k, want_scores=True)
            bits = torch.full_like(ref_bits, -1)
            scores = torch.full_like(ref_scores, float("nan"))
            out_bits, _ = binding.wide_route_static(ctx, x, wr, NG, k, mask_bits=bits, scores=scores)
            torch.cuda.synchronize()
            assert torch.equal(out_bits, ref_bits)
            oracle_mask = wo.mask_topk(wo.route_scores(host["x"], host["w_router"]), k)
            assert (bits_to_host(out_bits) == wo.pack_mask_bits(oracle_mask)).all()
            np.testing.assert_allclose(scores.cpu().numpy(), ref_scores.cpu().numpy(), rtol=1e-6, atol=1e-6)
            assert int(out_bits.cpu().numpy().view(np.uint32).astype(np.uint64).sum()) > 0
        assert ctx.status() == 0
    finally:
        ctx.close()


def test_static_route_pair_mode_and_size_limit():
    from paper_2607_28418_b200 import binding
    ctx = binding.Context(0)
    try:
        cfg = synth.CONFIGS["tiny"].with_(dtype="bf16")
        c = synth.make_ffn_case(cfg, 3)
        pr = synth.make_pair_router(cfg, 3, rank=16)
        x, w1, w2 = to_dev(c["x"], "bf16"), to_dev(pr["w1"], "bf16"), to_dev(pr["w2"], "bf16")
        ref_bits, _ = binding.wide_route(ctx, x, w1, cfg.n_groups, mode=binding.ROUTE_PAIR_ARGMAX, w2=w2, rank=16)
        bits, _ = binding.wide_route_static(ctx, x, w1, cfg.n_groups, mode=binding.ROUTE_PAIR_ARGMAX, w2=w2, rank=16)
        assert torch.equal(bits, ref_bits)
        oracle_mask = wo.mask_pair_argmax(wo.route_logits_pair(c["x"], pr["w1"], pr["w2"]))
        assert (bits_to_host(bits) == wo.pack_mask_bits(oracle_mask)).all()
        # 4096 tokens x 256 groups needs 16 MiB of scratch: beyond the fixed 2 MiB, must be refused
        big_x = torch.zeros((4096, 64), dtype=torch.bfloat16, device="cuda")
        big_w = torch.zeros((256, 64), dtype=torch.bfloat16, device="cuda")
        sentinel = torch.full((4096, 8), 7, dtype=torch.int32, device="cuda")
        with pytest.raises(binding.WideError) as e:
            binding.wide_route_static(ctx, big_x, big_w, 256, 128, mask_bits=sentinel)
        assert e.value.code == binding.ERR_WORKSPACE
        assert (sentinel == 7).all().item()          # nothing was launched
        assert ctx.status() == 0
    finally:
        ctx.close()
