"""GPU parity of the one-launch router for decode batches (at most 64 tokens, top-k mode, bf16): masks
bit for bit against the oracle's fp64 decision, beside the tensor-core form that larger batches take.

Covers token counts around the eight-token tiles, every mask-word count up to 256 groups, the layer
sizes of the decode workloads, weights built so that scores tie exactly or differ by one bf16 ulp
(the band around the selection boundary and its exact re-scoring decide those), per-token budgets
including 0 and all, the diagnostic scores, and repeated calls (the tickets of the tiles are shared
state every call must put back).
"""
import numpy as np
import pytest
import torch

from oracle import wide_oracle as wo
from paper_2607_28418_b200 import synth
from tests.gpu_util import bits_to_host, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_28418_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


def _check(ctx, x, wr, k, k_per_token=None, both=True):
    from paper_2607_28418_b200 import binding
    NG = wr.shape[0]
    s_ref = wo.route_scores(x, wr)
    ref = wo.pack_mask_bits(wo.mask_topk(s_ref, k if k_per_token is None else k_per_token))
    kt = None if k_per_token is None else torch.from_numpy(k_per_token.astype(np.int32)).cuda()
    xd, wd = to_dev(x, "bf16"), to_dev(wr, "bf16")
    bits, scores = binding.wide_route(ctx, xd, wd, NG, k, k_per_token=kt, want_scores=True)
    assert (bits_to_host(bits) == ref).all(), "one-launch form"
    if both:
        bits2, _ = binding.wide_route(ctx, xd, wd, NG, k, k_per_token=kt, flags=binding.FLAG_FORCE_PREFILL)
        assert torch.equal(bits, bits2), "tensor-core form"
    torch.cuda.synchronize()
    assert ctx.status() == 0
    return scores.cpu().numpy().astype(np.float64), s_ref


@pytest.mark.parametrize("T", [1, 2, 7, 8, 9, 33, 64])
@pytest.mark.parametrize("D,NG,k", [(4096, 112, 56), (5120, 108, 54), (1024, 224, 56), (512, 256, 100), (256, 33, 5), (64, 10, 5)])
def test_route_small_bit_exact(ctx, T, D, NG, k):
    rng = np.random.default_rng(1000 * T + NG)
    x = synth.make_activations(rng, T, D, "bf16", "random")
    wr = synth.make_weight(rng, NG, D, 1.0 / np.sqrt(D), "bf16")
    got, s_ref = _check(ctx, x, wr, k)
    # fp32 sums of D/32-long chains and five shuffle additions: inside the bound the band is built on
    eps = 2.0 ** -23 * (D / 32 + 8) * np.linalg.norm(x, axis=1, keepdims=True) * np.linalg.norm(wr, axis=1).max()
    assert (np.abs(got - s_ref) <= eps).all()


@pytest.mark.parametrize("T", [5, 64])
def test_route_small_exact_ties_and_one_ulp_rows(ctx, T):
    """All groups tie exactly except every third, which differs by one bf16 ulp in one weight: the
    fp32 scores cannot order those, the band and its fp64 re-scoring must."""
    D, NG, k = 1024, 96, 48
    rng = np.random.default_rng(42 + T)
    x = synth.round_to_bf16(rng.standard_normal((T, D)).astype(np.float32))
    base = synth.round_to_bf16((rng.standard_normal((1, D)) / np.sqrt(D)).astype(np.float32))
    wr = np.repeat(base, NG, axis=0)
    for g in range(0, NG, 3):
        i = int(rng.integers(0, D))
        wr[g, i] = synth.round_to_bf16(np.array([wr[g, i] * (1 + 2.0 ** -7)], dtype=np.float32))[0]
    _check(ctx, x, synth.round_to_bf16(wr), k)


def test_route_small_integer_ties_zero_row_and_per_token_budgets(ctx):
    T, D, NG = 40, 64, 20
    rng = np.random.default_rng(0)
    x = synth.round_to_bf16(rng.integers(-2, 3, size=(T, D)).astype(np.float32))   # many exact ties
    x[0] = 0.0
    wr = synth.round_to_bf16(rng.integers(-1, 2, size=(NG, D)).astype(np.float32))
    kt = rng.integers(0, NG + 1, size=T)
    kt[1], kt[2] = 0, NG
    _check(ctx, x, wr, 0, k_per_token=kt)
    for k in (0, 1, NG - 1, NG):
        _check(ctx, x, wr, k)


def test_route_small_repeated_calls_of_different_sizes(ctx):
    """The tickets of the token tiles go back to zero with every call: a call with eight tiles, then one
    with a single tile, then eight again, each twice, must all decide like the oracle."""
    rng = np.random.default_rng(7)
    D, NG, k = 2048, 112, 56
    wr = synth.make_weight(rng, NG, D, 1.0 / np.sqrt(D), "bf16")
    for T in (64, 1, 64, 3, 17, 17, 1, 64):
        x = synth.make_activations(rng, T, D, "bf16", "random")
        _check(ctx, x, wr, k, both=False)


@pytest.mark.parametrize("T", [3, 40])
def test_route_small_band_rescoring_with_a_wide_range_of_magnitudes(ctx, T):
    """Rows that tie exactly or differ by one ulp put most groups in the band, whose members are re-scored
    exactly; a few elements of x and of the weights are tiny (2^-100, 2^-60) or large (2^20), so that the
    products of one row span a hundred binary orders of magnitude.  The decision must stay the oracle's."""
    D, NG, k = 1024, 64, 32
    rng = np.random.default_rng(77 + T)
    x = synth.round_to_bf16(rng.standard_normal((T, D)).astype(np.float32))
    base = synth.round_to_bf16((rng.standard_normal((1, D)) / np.sqrt(D)).astype(np.float32))
    wr = np.repeat(base, NG, axis=0)
    for g in range(0, NG, 3):
        i = int(rng.integers(0, D))
        wr[g, i] = synth.round_to_bf16(np.array([wr[g, i] * (1 + 2.0 ** -7)], dtype=np.float32))[0]
    wr[5, 7] = np.float32(2.0 ** -60)
    wr[6, 9] = np.float32(2.0 ** -100)
    for t in range(T):
        if t % 3 == 1:
            x[t, t % D] = np.float32(2.0 ** -100)
        if t % 3 == 2:
            x[t, (5 * t) % D] = np.float32(2.0 ** 20)
    _check(ctx, synth.round_to_bf16(x), synth.round_to_bf16(wr), k)
