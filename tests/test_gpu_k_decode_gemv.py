"""GPU parity of the matrix-vector decode kernel (one or two tokens: the GEMV dispatch for tiny M of
Appendix B) behind wide_ffn and wide_oproj, against the oracle and beside the tensor-core decode kernel.

Covers both token counts, every group size, both output types, a hidden size whose rows are not a
whole number of 32-piece sweeps, a token with nothing active (its row is exactly zero and it adds
nothing to the union), the all-zero and the all-ones mask, the O-projection form (no first pass, no
barrier), repeated and interleaved calls on one context (the barrier words and the channel pool's
counter are shared state that every call must leave clean) and the no-op contract after an expired wait.
"""
import numpy as np
import pytest
import torch

from oracle import wide_oracle as wo
from paper_2607_28418_b200 import synth
from tests.gpu_util import assert_close, bits_to_dev, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_28418_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


def _ffn(ctx, B, D, Dff, G, mask, flags, out=None, seed=0):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=B, hidden=D, d_ff=Dff, group=G, k=1)
    case = synth.make_ffn_case(cfg, seed)
    ref = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"], mask, G)
    dev = {n: to_dev(case[n], "bf16") for n in ("x", "w_gate", "w_up", "w_down")}
    ctx.workspace(1 << 20).fill_(0xFF)      # stale scratch must not leak into the result
    y = binding.wide_ffn(ctx, dev["x"], dev["w_gate"], dev["w_up"], dev["w_down"], G, bits_to_dev(wo.pack_mask_bits(mask)),
                         None, out_dtype=out, flags=flags)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    return y, ref


@pytest.mark.parametrize("out", [None, torch.float32])
@pytest.mark.parametrize("G", [64, 128, 256, 512])
@pytest.mark.parametrize("B", [1, 2])
def test_ffn_gemv_and_tensor_core_kernel_match_the_oracle(ctx, B, G, out):
    from paper_2607_28418_b200 import binding
    assert B <= binding.DECODE_GEMV_MAX_TOKENS
    D, Dff = 1024, 4096
    mask = synth.random_mask(100 * B + G, B, Dff // G, max(1, Dff // G // 2))
    for name, flags in (("gemv", binding.FLAG_NONE), ("tensor-core", binding.FLAG_DECODE_TC)):
        y, ref = _ffn(ctx, B, D, Dff, G, mask, flags, out=out, seed=B + G)
        assert_close(y, ref, f"{name} B{B} G{G} out {out}")


@pytest.mark.parametrize("D,Dff,G", [(320, 1280, 64), (576, 2304, 128), (4096, 14336, 128), (5120, 13824, 128)])
def test_ffn_gemv_rows_that_are_not_whole_sweeps(ctx, D, Dff, G):
    """hidden / 8 = 40 or 72 pieces per row (not a multiple of the 32 lanes, nor of a 128-piece batch),
    unions whose W_down pieces do not fill the last batch; and the full Llama-3-8B and Llama-2-13B shapes."""
    from paper_2607_28418_b200 import binding
    for B in (1, 2):
        mask = synth.random_mask(7 * B + D, B, Dff // G, 3 if D < 4096 else Dff // G // 2)
        y, ref = _ffn(ctx, B, D, Dff, G, mask, binding.FLAG_NONE, seed=D + B)
        assert_close(y, ref, f"B{B} D{D} Dff{Dff} G{G}")


def test_ffn_gemv_closed_cases(ctx):
    from paper_2607_28418_b200 import binding
    D, Dff, G = 512, 2048, 128
    NG = Dff // G
    # a token with nothing active beside one with a budget of its own
    mask = np.zeros((2, NG), dtype=bool)
    mask[0, [1, 5, 6, 15]] = True
    y, ref = _ffn(ctx, 2, D, Dff, G, mask, binding.FLAG_NONE, seed=3)
    assert_close(y, ref, "one empty token")
    assert (y[1] == 0).all().item()
    # nothing active at all: exact zeros, no barrier, no pool
    y, _ = _ffn(ctx, 2, D, Dff, G, np.zeros((2, NG), dtype=bool), binding.FLAG_NONE, seed=3)
    assert (y == 0).all().item()
    # everything active: the dense FFN
    for B in (1, 2):
        y, ref = _ffn(ctx, B, D, Dff, G, np.ones((B, NG), dtype=bool), binding.FLAG_NONE, out=torch.float32, seed=4)
        assert_close(y, ref, f"dense B{B}")
    # disjoint masks: the union is the sum of the two, each token must still see only its own groups
    mask = np.zeros((2, NG), dtype=bool)
    mask[0, :NG // 2] = True
    mask[1, NG // 2:] = True
    y, ref = _ffn(ctx, 2, D, Dff, G, mask, binding.FLAG_NONE, seed=5)
    assert_close(y, ref, "disjoint masks")


@pytest.mark.parametrize("B", [1, 2])
@pytest.mark.parametrize("G,K", [(512, 2048), (128, 1024), (64, 512)])
def test_oproj_gemv_and_tensor_core_kernel_match_the_oracle(ctx, B, G, K):
    from paper_2607_28418_b200 import binding
    D = 768
    rng = np.random.default_rng(B + G)
    a = synth.make_activations(rng, B, K, "bf16", "random")
    w_o = synth.make_weight(rng, D, K, 0.02, "bf16")
    mask = synth.random_mask(B + K, B, K // G, max(1, K // G // 2))
    if B == 2:
        mask[1] = False
        mask[1, 0] = True          # budgets differ between the tokens
    ref = wo.oproj(a, w_o, mask, G)
    for name, flags in (("gemv", binding.FLAG_NONE), ("tensor-core", binding.FLAG_DECODE_TC)):
        y = binding.wide_oproj(ctx, to_dev(a, "bf16"), to_dev(w_o, "bf16"), G, bits_to_dev(wo.pack_mask_bits(mask)), None,
                               flags=flags)
        torch.cuda.synchronize()
        assert ctx.status() == 0
        assert_close(y, ref, f"oproj {name} B{B} G{G}")


def test_interleaved_calls_leave_the_shared_words_clean_and_results_repeat(ctx):
    """GEMV and tensor-core decode calls share the context's barrier words; the GEMV kernel also draws
    channels from a counter that the call itself must put back.  Any order of calls, any shapes."""
    from paper_2607_28418_b200 import binding
    seq = [(1, 1024, 4096, 128, 0), (8, 512, 2048, 128, 0), (2, 512, 2048, 64, 0), (2, 512, 2048, 64, binding.FLAG_DECODE_TC),
           (1, 1024, 4096, 128, 0), (1, 320, 1280, 64, 0), (64, 512, 2048, 256, 0), (2, 1024, 4096, 512, 0)]
    first = {}
    for i, (B, D, Dff, G, flags) in enumerate(seq):
        mask = synth.random_mask(B + D + G, B, Dff // G, max(1, Dff // G // 2))
        y, ref = _ffn(ctx, B, D, Dff, G, mask, flags, seed=B + D)
        assert_close(y, ref, f"call {i}: B{B} D{D} Dff{Dff} G{G} flags {flags}")
        key = (B, D, Dff, G, flags)
        if key in first:
            assert torch.equal(first[key], y), "the same call twice must give the same bits"
        first[key] = y.clone()


def test_gemv_call_is_a_no_op_until_the_status_is_read():
    from paper_2607_28418_b200 import binding
    ctx = binding.Context(0)
    try:
        D, Dff, G = 512, 1024, 128
        cfg = synth.WideConfig("dirty", tokens=1, hidden=D, d_ff=Dff, group=G, k=4)
        case = synth.make_ffn_case(cfg, 6)
        dev = {k: to_dev(v, "bf16") for k, v in case.items()}
        mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router"]), cfg.k)
        bits = bits_to_dev(wo.pack_mask_bits(mask))
        ctx.set_wait_limit_ns(2_000_000)
        ctx.selftest_wait()                                     # sets the status word, never read here
        y = torch.full((1, D), 7.0, dtype=torch.bfloat16, device="cuda")
        binding.wide_ffn(ctx, dev["x"], dev["w_gate"], dev["w_up"], dev["w_down"], G, bits, None, y=y)
        torch.cuda.synchronize()
        assert (y == 7.0).all().item()                          # nothing was written
        assert ctx.status() == binding.ERR_TIMEOUT
        ctx.set_wait_limit_ns(2_000_000_000)
        binding.wide_ffn(ctx, dev["x"], dev["w_gate"], dev["w_up"], dev["w_down"], G, bits, None, y=y)
        ref = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"], mask, G)
        assert_close(y, ref, "after the status was read")
        assert ctx.status() == 0
    finally:
        ctx.close()
