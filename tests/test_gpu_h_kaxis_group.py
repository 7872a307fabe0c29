"""GPU parity of the per-group K-axis kernel (Eq. 10 / Algorithm 3: active (tile, group) blocks only,
partial sums scatter-reduced into the output) behind wide_oproj and wide_ffn, against the oracle.

Covers every reduction variant (fp32 sums straight into an fp32 output, fp32 sums in scratch
converted to bf16, bf16 sums straight into a bf16 output), group sizes 64..512, output widths that
are not a multiple of the 256-column block, ragged row tiles, masks with a variable budget, a token
with nothing active, a group nobody selects, stale scratch, and the choice between the two K-axis
kernels that the kernels take on the device.
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


def _oproj(ctx, T, D, K, G, mask, flags, out_dtype=None, seed=0):
    from paper_2607_28418_b200 import binding
    rng = np.random.default_rng(seed)
    a = synth.make_activations(rng, T, K, "bf16", "random")
    w_o = synth.make_weight(rng, D, K, 0.02, "bf16")
    ref = wo.oproj(a, w_o, mask, G)
    ctx.workspace(1 << 20).fill_(0xFF)      # stale scratch must not leak into the sums
    y = binding.wide_oproj(ctx, to_dev(a, "bf16"), to_dev(w_o, "bf16"), G, bits_to_dev(wo.pack_mask_bits(mask)),
                           meta_to_dev(wo.reorder(mask, 128)), out_dtype=out_dtype, flags=flags)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    return y, ref


@pytest.mark.parametrize("out", [None, torch.float32])
@pytest.mark.parametrize("T,D,K,G,k", [(300, 512, 1024, 512, 1), (700, 1024, 2048, 256, 3), (130, 512, 512, 64, 4),
                                       (1000, 768, 1024, 128, 5), (513, 640, 1536, 512, 2), (129, 320, 2048, 64, 9)])
def test_oproj_per_group_kernel(ctx, T, D, K, G, k, out):
    """Forced per-group kernel.  bf16 output: bf16 sums for up to 16 groups, fp32 scratch + convert
    for the 32-group shape; fp32 output: fp32 sums in the output itself."""
    from paper_2607_28418_b200 import binding
    mask = synth.random_mask(T + K + G, T, K // G, k)
    y, ref = _oproj(ctx, T, D, K, G, mask, binding.FLAG_FORCE_PREFILL | binding.FLAG_KAXIS_GROUP, out_dtype=out, seed=T)
    assert_close(y, ref, f"oproj per-group {T}x{D}x{K} G{G} out {out}")


def test_oproj_per_group_variable_budget_and_empty_rows(ctx):
    from paper_2607_28418_b200 import binding
    T, D, K, G = 900, 512, 2048, 256
    mask = synth.bernoulli_mask(5, T, K // G, 0.4)
    mask[:, 3] = False       # a group nobody selects: no item at all
    mask[:, 5] = True        # a group everybody selects: 7 full tiles and a ragged one
    mask[7] = False          # a token with nothing active: its output row is exactly zero
    for out in (None, torch.float32):
        y, ref = _oproj(ctx, T, D, K, G, mask, binding.FLAG_FORCE_PREFILL | binding.FLAG_KAXIS_GROUP, out_dtype=out, seed=3)
        assert_close(y, ref, f"variable budget, out {out}")
        assert (y[7] == 0).all().item()


def test_oproj_bf16_sums_on_request(ctx):
    """32 groups would sum in fp32 scratch by default; WIDE_FLAG_REDUCE_BF16 adds in bf16 instead."""
    from paper_2607_28418_b200 import binding
    T, D, K, G, k = 400, 512, 2048, 64, 12
    mask = synth.random_mask(77, T, K // G, k)
    flags = binding.FLAG_FORCE_PREFILL | binding.FLAG_KAXIS_GROUP
    y32, ref = _oproj(ctx, T, D, K, G, mask, flags, seed=9)
    y16, _ = _oproj(ctx, T, D, K, G, mask, flags | binding.FLAG_REDUCE_BF16, seed=9)
    e32 = assert_close(y32, ref, "fp32 sums")
    e16 = assert_close(y16, ref, "bf16 sums")
    print(f"rel err fp32 sums {e32:.2e}, bf16 sums {e16:.2e}")


@pytest.mark.parametrize("k", [1, 2, 4])
def test_oproj_choice_on_the_device_gives_the_same_result_either_way(ctx, k):
    """group 512: the kernels choose by the padded active fraction (1 of 4 groups: per-group kernel,
    all 4: owner-computes).  Either way the output must match the oracle and the forced variants."""
    from paper_2607_28418_b200 import binding
    T, D, K, G = 1100, 512, 2048, 512
    mask = synth.random_mask(k, T, K // G, k)
    auto, ref = _oproj(ctx, T, D, K, G, mask, binding.FLAG_FORCE_PREFILL, seed=k)
    grp, _ = _oproj(ctx, T, D, K, G, mask, binding.FLAG_FORCE_PREFILL | binding.FLAG_KAXIS_GROUP, seed=k)
    own, _ = _oproj(ctx, T, D, K, G, mask, binding.FLAG_FORCE_PREFILL | binding.FLAG_KAXIS_OWNER, seed=k)
    for name, y in (("auto", auto), ("per-group", grp), ("owner", own)):
        assert_close(y, ref, f"k={k} {name}")


def test_oproj_masked_input_per_group(ctx):
    from paper_2607_28418_b200 import binding
    T, D, K, G, k = 700, 512, 1024, 256, 2
    rng = np.random.default_rng(8)
    a = synth.make_activations(rng, T, K, "bf16", "random")
    w_o = synth.make_weight(rng, D, K, 0.02, "bf16")
    mask = synth.random_mask(9, T, K // G, k)
    a_masked = (a * wo.expand_group_mask(mask, G)).astype(np.float32)
    for flags in (binding.FLAG_INPUT_MASKED, binding.FLAG_INPUT_MASKED | binding.FLAG_KAXIS_GROUP):
        y = binding.wide_oproj(ctx, to_dev(a_masked, "bf16"), to_dev(w_o, "bf16"), G, bits_to_dev(wo.pack_mask_bits(mask)),
                               meta_to_dev(wo.reorder(mask, 128)), flags=flags)
        assert_close(y, wo.oproj(a, w_o, mask, G), f"masked input, flags {flags}")
    assert ctx.status() == 0


@pytest.mark.parametrize("T,D,Dff,G,k,router,out", [(640, 1024, 2048, 128, 8, "random", None),
                                                    (700, 512, 4096, 128, 8, "clustered", None),
                                                    (300, 512, 2048, 256, 2, "random", torch.float32),
                                                    (257, 512, 1024, 64, 4, "random", None)])
def test_ffn_down_projection_per_group(ctx, T, D, Dff, G, k, router, out):
    """wide_ffn with the down projection forced to the per-group kernel: gate/up scatters H in
    (clustered) token order, the per-group kernel gathers the active rows back through the
    permutation."""
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=T, hidden=D, d_ff=Dff, group=G, k=k, router=router)
    case = synth.make_ffn_case(cfg, 31)
    mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router"]), k)
    ref = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"], mask, G)
    dev = {n: to_dev(case[n], "bf16") for n in ("x", "w_gate", "w_up", "w_down")}
    ctx.workspace(1 << 20).fill_(0xFF)
    y = binding.wide_ffn(ctx, dev["x"], dev["w_gate"], dev["w_up"], dev["w_down"], G, bits_to_dev(wo.pack_mask_bits(mask)),
                         meta_to_dev(wo.reorder(mask, 128)), out_dtype=out,
                         flags=binding.FLAG_FORCE_PREFILL | binding.FLAG_KAXIS_GROUP)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    assert_close(y, ref, f"ffn per-group down {T}x{D}x{Dff} G{G}")


def test_flag_combinations_are_validated_on_the_host(ctx):
    from paper_2607_28418_b200 import binding
    T, D, K, G = 256, 256, 512, 256
    a = torch.zeros((T, K), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((D, K), dtype=torch.bfloat16, device="cuda")
    bits = torch.zeros((T, 1), dtype=torch.int32, device="cuda")
    meta = meta_to_dev(wo.reorder(np.zeros((T, 2), dtype=bool), 128))
    with pytest.raises(binding.WideError) as e:
        binding.wide_oproj(ctx, a, w, G, bits, meta, flags=binding.FLAG_KAXIS_GROUP | binding.FLAG_KAXIS_OWNER)
    assert e.value.code == binding.ERR_INVALID_ARG
    with pytest.raises(binding.WideError) as e:      # the per-group kernel needs the permutation
        binding.wide_oproj(ctx, a, w, G, bits, None, flags=binding.FLAG_FORCE_PREFILL | binding.FLAG_KAXIS_GROUP)
    assert e.value.code == binding.ERR_INVALID_ARG


def test_per_group_kernel_narrow_output_and_empty_batch(ctx):
    """An output narrower than one 256-column block, and a call with no tokens at all."""
    from paper_2607_28418_b200 import binding
    T, D, K, G, k = 200, 128, 1024, 256, 2
    mask = synth.random_mask(4, T, K // G, k)
    y, ref = _oproj(ctx, T, D, K, G, mask, binding.FLAG_FORCE_PREFILL | binding.FLAG_KAXIS_GROUP, seed=2)
    assert_close(y, ref, "hidden 128")
    # an empty batch, through the C ABI itself (torch hands out null pointers for empty tensors, and
    # the entry points refuse null pointers): nothing is launched, the output is left alone
    import ctypes
    a = torch.zeros((1, K), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((D, K), dtype=torch.bfloat16, device="cuda")
    small = torch.zeros((8,), dtype=torch.int32, device="cuda")
    y0 = torch.full((1, D), 3.0, dtype=torch.bfloat16, device="cuda")
    ws = ctx.workspace(1 << 20)
    vp = lambda t: ctypes.c_void_p(t.data_ptr())
    rc = ctx.lib.wide_oproj(ctx.handle, ctypes.c_void_p(torch.cuda.current_stream().cuda_stream), vp(a), vp(w), binding.BF16,
                            0, D, K, G, vp(small), vp(small), vp(small), None, None, vp(y0), binding.BF16, vp(ws), ws.numel(),
                            binding.FLAG_FORCE_PREFILL | binding.FLAG_KAXIS_GROUP)
    torch.cuda.synchronize()
    assert rc == 0 and (y0 == 3.0).all().item() and ctx.status() == 0
