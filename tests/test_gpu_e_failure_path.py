"""The bounded-wait failure path: a wait that can never be satisfied gives up after the context's
bound, the host reads WIDE_ERR_TIMEOUT, and the context keeps working.  Nothing faults or hangs."""
import numpy as np
import pytest
import torch

from oracle import wide_oracle as wo
from paper_2607_28418_b200 import synth
from tests.gpu_util import bits_to_host, to_dev

pytestmark = pytest.mark.gpu


def test_expired_wait_sets_status_and_context_survives():
    from paper_2607_28418_b200 import binding
    ctx = binding.Context(0)
    try:
        assert ctx.status() == 0
        ctx.set_wait_limit_ns(3_000_000)                       # 3 ms
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.selftest_wait()
        e1.record()
        torch.cuda.synchronize()
        assert 2.5 <= e0.elapsed_time(e1) < 500.0              # gave up after the bound, not before
        assert ctx.status() == binding.ERR_TIMEOUT
        assert ctx.status() == 0                               # reading clears it
        ctx.set_wait_limit_ns(2_000_000_000)
        # the same context still routes and runs a decode FFN correctly (its buffers were reset)
        cfg = synth.WideConfig("after_timeout", tokens=16, hidden=512, d_ff=1024, group=128, k=4)
        case = synth.make_ffn_case(cfg, 5)
        dev = {k: to_dev(v, cfg.dtype) for k, v in case.items()}
        bits, _ = binding.wide_route(ctx, dev["x"], dev["w_router"], cfg.n_groups, cfg.k)
        mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router"]), cfg.k)
        assert (bits_to_host(bits) == wo.pack_mask_bits(mask)).all()
        y = binding.wide_ffn(ctx, dev["x"], dev["w_gate"], dev["w_up"], dev["w_down"], cfg.group, bits, None)
        ref = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"], mask, cfg.group)
        assert np.abs(y.float().cpu().numpy() - ref).max() <= 2e-2 * np.abs(ref).max()
        assert ctx.status() == 0
    finally:
        ctx.close()


def test_decode_calls_are_no_ops_until_the_status_is_read():
    """After a wait has expired the decode path's counters and sums may be dirty; until
    wide_status resets them a decode call must leave its output alone instead of adding to them."""
    from paper_2607_28418_b200 import binding
    ctx = binding.Context(0)
    try:
        cfg = synth.WideConfig("dirty", tokens=8, hidden=512, d_ff=1024, group=128, k=4)
        case = synth.make_ffn_case(cfg, 6)
        dev = {k: to_dev(v, cfg.dtype) for k, v in case.items()}
        mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router"]), cfg.k)
        bits = torch.from_numpy(wo.pack_mask_bits(mask).view(np.int32)).cuda()
        ctx.set_wait_limit_ns(2_000_000)
        ctx.selftest_wait()                                     # sets the status word, never read here
        y = torch.full((8, 512), 7.0, dtype=torch.bfloat16, device="cuda")
        binding.wide_ffn(ctx, dev["x"], dev["w_gate"], dev["w_up"], dev["w_down"], cfg.group, bits, None, y=y)
        torch.cuda.synchronize()
        assert (y == 7.0).all().item()                          # nothing was written
        assert ctx.status() == binding.ERR_TIMEOUT
        ctx.set_wait_limit_ns(2_000_000_000)
        binding.wide_ffn(ctx, dev["x"], dev["w_gate"], dev["w_up"], dev["w_down"], cfg.group, bits, None, y=y)
        ref = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"], mask, cfg.group)
        assert np.abs(y.float().cpu().numpy() - ref).max() <= 2e-2 * np.abs(ref).max()
        assert ctx.status() == 0
    finally:
        ctx.close()
