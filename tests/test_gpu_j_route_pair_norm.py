"""GPU parity of wide_route_pair_prepare / wide_route_pair_norm (Eq. 4 on the RMSNorm of the hidden
state, weight-only work prepared once) against the oracle: masks bit for bit, logits within fp32
round-off, including exact ties, pairs one bf16 ulp apart and an all-zero token."""
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


def _router(rng, D, rank, NG, gamma_std=0.1):
    w1 = synth.round_to_bf16((rng.standard_normal((D, rank)) / np.sqrt(D)).astype(np.float32))
    w2 = synth.round_to_bf16((rng.standard_normal((rank, NG, 2)) / np.sqrt(rank)).astype(np.float32))
    gamma = synth.round_to_bf16((1.0 + gamma_std * rng.standard_normal(D)).astype(np.float32))
    return w1, w2, gamma


def _run(ctx, x, w1, w2, gamma, eps, NG, want_scores=True):
    from paper_2607_28418_b200 import binding
    w1d, w2d = to_dev(w1, "bf16"), to_dev(w2, "bf16")
    gd = None if gamma is None else to_dev(gamma, "bf16")
    prepared = binding.wide_route_pair_prepare(ctx, w1d, w2d, gd, NG)
    bits, scores = binding.wide_route_pair_norm(ctx, to_dev(x, "bf16"), w1d, w2d, gd, eps, prepared, NG, want_scores=want_scores)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    return bits, scores, (w1d, w2d, gd, prepared)


@pytest.mark.parametrize("T,D,NG,rank", [(1024, 2048, 86, 16), (8, 4096, 192, 32), (300, 1024, 10, 8), (2048, 4096, 86, 16)])
def test_pair_norm_layer_size_and_near_ties(ctx, T, D, NG, rank):
    rng = np.random.default_rng(T + NG)
    x = synth.round_to_bf16((rng.standard_normal((T, D)) * rng.uniform(0.2, 5.0, size=(T, 1))).astype(np.float32))
    x[3] = 0.0                                                      # every pair ties: everything executes
    w1, w2, gamma = _router(rng, D, rank, NG)
    w2[:, 0::5, 1] = w2[:, 0::5, 0]                                 # exact ties for every token
    for g in range(1, NG, 5):                                       # one ulp apart in one row
        c = int(rng.integers(0, rank))
        w2[:, g, 1] = w2[:, g, 0]
        w2[c, g, 1] = synth.round_to_bf16(np.array([w2[c, g, 0] * (1 + 2.0 ** -7)], dtype=np.float32))[0]
    w2 = synth.round_to_bf16(w2).reshape(rank, 2 * NG)
    eps = 1e-5
    logits = wo.route_logits_pair_norm(x, gamma, eps, w1, w2)
    ref = wo.pack_mask_bits(wo.mask_pair_argmax(logits))
    bits, scores, _ = _run(ctx, x, w1, w2, gamma, eps, NG)
    assert (bits_to_host(bits) == ref).all()
    assert (bits_to_host(bits)[3] == wo.pack_mask_bits(np.ones((1, NG), dtype=bool))[0]).all()
    np.testing.assert_allclose(scores.cpu().numpy(), logits.reshape(T, -1), rtol=2e-3, atol=2e-3)


def test_pair_norm_exact_arithmetic_ties(ctx):
    """Inputs on which every sum is exact in fp64 (tokens of +-1: rms = 1 with eps = 0; norm weights
    that are powers of two; small integer router weights), so that the many pairs that tie do so in
    the oracle's arithmetic as well."""
    T, D, NG, rank = 256, 256, 40, 8
    rng = np.random.default_rng(3)
    x = (2.0 * rng.integers(0, 2, size=(T, D)) - 1.0).astype(np.float32)
    gamma = np.array([0.5, 1.0, 2.0], dtype=np.float32)[rng.integers(0, 3, size=D)]
    w1 = rng.integers(-1, 2, size=(D, rank)).astype(np.float32)
    w2 = rng.integers(-1, 2, size=(rank, 2 * NG)).astype(np.float32)
    logits = wo.route_logits_pair_norm(x, gamma, 0.0, w1, w2)
    assert (logits[:, :, 0] == logits[:, :, 1]).sum() >= 20         # there are real ties in here
    bits, _, _ = _run(ctx, x, w1, w2, gamma, 0.0, NG, want_scores=False)
    assert (bits_to_host(bits) == wo.pack_mask_bits(wo.mask_pair_argmax(logits))).all()


def test_pair_norm_ignores_the_row_scale_and_matches_the_plain_pair_router(ctx):
    from paper_2607_28418_b200 import binding
    T, D, NG, rank = 700, 1024, 86, 16
    rng = np.random.default_rng(5)
    x = synth.round_to_bf16(rng.standard_normal((T, D)).astype(np.float32))
    w1, w2, _ = _router(rng, D, rank, NG)
    w2 = w2.reshape(rank, 2 * NG)
    bits, _, (w1d, w2d, _, prepared) = _run(ctx, x, w1, w2, None, 1e-6, NG, want_scores=False)
    # no norm weight: the decision is the one of the plain Eq. 4 router on x itself
    plain, _ = binding.wide_route(ctx, to_dev(x, "bf16"), w1d, NG, mode=binding.ROUTE_PAIR_ARGMAX, w2=w2d, rank=rank)
    assert torch.equal(bits, plain)
    # a token scaled by a power of two (exact in bf16) routes the same way; the prepared buffer is reused
    scaled, _ = binding.wide_route_pair_norm(ctx, to_dev(x * 4.0, "bf16"), w1d, w2d, None, 1e-6, prepared, NG)
    assert torch.equal(bits, scaled)


def test_pair_norm_argument_errors(ctx):
    from paper_2607_28418_b200 import binding
    w1 = torch.zeros((256, 12), dtype=torch.bfloat16, device="cuda")       # rank 12: not a multiple of 8
    w2 = torch.zeros((12, 16), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.WideError) as e:
        binding.wide_route_pair_prepare(ctx, w1, w2, None, 8)
    assert e.value.code == binding.ERR_UNSUPPORTED_SHAPE
