"""Parity of wide_attn (masked FlashAttention prefill, Algorithm 4) with the oracle."""
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


def _run(ctx, case, mask, h_q, h_kv, d, hpg, causal=True, scale=0.0):
    from paper_2607_28418_b200 import binding
    t_q, t_k = case["q"].shape[0], case["k"].shape[0]
    meta = meta_to_dev(wo.reorder(mask, 128))     # stage-wise: the oracle's permutation goes in
    o = binding.wide_attn(ctx, to_dev(case["q"].reshape(t_q, h_q * d), "bf16"), to_dev(case["k"].reshape(t_k, h_kv * d), "bf16"),
                          to_dev(case["v"].reshape(t_k, h_kv * d), "bf16"), h_q, h_kv, hpg, meta, causal=causal, scale=scale)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    return o.reshape(t_q, h_q, d)


@pytest.mark.parametrize("t_q,t_k,h_q,h_kv,d,hpg,p", [
    (128, 128, 4, 4, 128, 2, 0.5),
    (300, 300, 8, 2, 128, 4, 0.5),       # GQA, ragged last tile
    (517, 517, 4, 4, 64, 1, 0.3),        # head_dim 64
    (200, 455, 4, 2, 128, 2, 0.7),       # keys ahead of the queries (delta > 0)
    (1024, 1024, 8, 8, 128, 4, 0.5),     # several key tiles per query tile
])
@pytest.mark.parametrize("causal", [True, False])
def test_attn_matches_oracle(ctx, t_q, t_k, h_q, h_kv, d, hpg, p, causal):
    case = synth.make_attn_case(3, t_q, t_k, h_q, h_kv, d)
    mask = synth.bernoulli_mask(5, t_q, h_q // hpg, p)
    got = _run(ctx, case, mask, h_q, h_kv, d, hpg, causal=causal)
    ref = wo.masked_attention(case["q"], case["k"], case["v"], mask, hpg, causal=causal)
    head_mask = np.repeat(mask, hpg, axis=1)
    assert (got.float().cpu().numpy()[~head_mask] == 0.0).all()   # inactive pairs: exact zeros
    assert_close(got, ref, "attn")


def test_attn_closed_cases(ctx):
    t, h_q, h_kv, d, hpg = 260, 4, 2, 128, 2
    case = synth.make_attn_case(9, t, t, h_q, h_kv, d)
    ones = np.ones((t, h_q // hpg), dtype=bool)
    zeros = np.zeros_like(ones)
    assert (_run(ctx, case, zeros, h_q, h_kv, d, hpg) == 0.0).all().item()
    # the same value vector at every key: every active output row is that vector
    case["v"][:] = synth.round_to_bf16(np.linspace(-1, 1, d).astype(np.float32))
    got = _run(ctx, case, ones, h_q, h_kv, d, hpg).float().cpu().numpy()
    np.testing.assert_allclose(got, np.broadcast_to(case["v"][0, 0], got.shape), atol=1e-2)
    # the first token attends to itself only
    case = synth.make_attn_case(10, t, t, h_q, h_kv, d)
    got = _run(ctx, case, ones, h_q, h_kv, d, hpg).float().cpu().numpy()
    np.testing.assert_allclose(got[0], np.repeat(case["v"][0], h_q // h_kv, axis=0), atol=1e-2)


def test_attn_one_group_active_per_token_and_custom_scale(ctx):
    t, h_q, h_kv, d, hpg = 384, 8, 4, 128, 2
    case = synth.make_attn_case(11, t, t, h_q, h_kv, d)
    mask = synth.random_mask(12, t, h_q // hpg, 1)
    got = _run(ctx, case, mask, h_q, h_kv, d, hpg, scale=0.05)
    ref = wo.masked_attention(case["q"], case["k"], case["v"], mask, hpg, scale=0.05)
    assert_close(got, ref, "attn, custom scale")


def test_attn_more_items_than_sms_with_uneven_groups(ctx):
    """The prefill kernel runs one CTA per SM and hands (head, query tile) items out at run time.  Here
    about 200 items of 1 to 20 key tiles go over the CTAs: three groups with every token, two with
    half, one with 90 %, one with 37 tokens, one with none (no item at all, rows of exact zeros)."""
    t, h_q, h_kv, d, hpg = 2560, 16, 4, 128, 2
    case = synth.make_attn_case(21, t, t, h_q, h_kv, d)
    rng = np.random.default_rng(22)
    mask = np.zeros((t, h_q // hpg), dtype=bool)
    mask[:, [0, 3, 5]] = True
    mask[:, 1] = rng.random(t) < 0.5
    mask[:, 6] = rng.random(t) < 0.5
    mask[rng.choice(t, 37, replace=False), 2] = True
    mask[:, 7] = rng.random(t) < 0.9
    got = _run(ctx, case, mask, h_q, h_kv, d, hpg)
    ref = wo.masked_attention(case["q"], case["k"], case["v"], mask, hpg)
    head_mask = np.repeat(mask, hpg, axis=1)
    assert (got.float().cpu().numpy()[~head_mask] == 0.0).all()
    assert_close(got, ref, "attn, more items than SMs")


def test_attn_queries_ahead_of_the_keys(ctx):
    """T_k < T_q with the causal limit j <= t + T_k - T_q: the first queries see no key at all (exact
    zero rows, whole query tiles without a key tile), the next ones a single, partly visible key tile."""
    t_q, t_k, h_q, h_kv, d, hpg = 600, 200, 4, 2, 128, 2
    case = synth.make_attn_case(23, t_q, t_k, h_q, h_kv, d)
    for mask in (synth.bernoulli_mask(24, t_q, h_q // hpg, 0.5), np.ones((t_q, h_q // hpg), dtype=bool)):
        got = _run(ctx, case, mask, h_q, h_kv, d, hpg)
        ref = wo.masked_attention(case["q"], case["k"], case["v"], mask, hpg)
        assert (got[: t_q - t_k] == 0.0).all().item()
        assert_close(got, ref, "attn, T_k < T_q")


def test_attn_repeated_and_interleaved_calls_repeat_bit_for_bit(ctx):
    """The work list's counter is shared state that every launch must leave at zero, whatever the shapes
    of the calls before; which CTA takes which item may differ from run to run, the bits may not."""
    shapes = [(300, 300, 8, 2, 128, 4), (1536, 1536, 16, 16, 128, 4), (517, 517, 4, 4, 64, 1)]
    first = {}
    for rep in range(3):
        for sh in shapes:
            t_q, t_k, h_q, h_kv, d, hpg = sh
            case = synth.make_attn_case(31, t_q, t_k, h_q, h_kv, d)
            mask = synth.bernoulli_mask(32, t_q, h_q // hpg, 0.6)
            got = _run(ctx, case, mask, h_q, h_kv, d, hpg)
            if sh in first:
                assert torch.equal(first[sh], got), f"{sh}: call {rep} differs from the first"
            else:
                first[sh] = got.clone()
                assert_close(got, wo.masked_attention(case["q"], case["k"], case["v"], mask, hpg), f"attn {sh}")


def test_attn_rejects_bad_arguments(ctx):
    from paper_2607_28418_b200 import binding
    q = torch.zeros((128, 4 * 96), dtype=torch.bfloat16, device="cuda")
    meta = meta_to_dev(wo.reorder(np.ones((128, 2), dtype=bool), 128))
    with pytest.raises(binding.WideError):
        binding.wide_attn(ctx, q, q, q, 4, 4, 2, meta)             # head_dim 96
    q = torch.zeros((128, 4 * 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.WideError):
        binding.wide_attn(ctx, q, q, q, 4, 3, 2, meta)             # heads not divisible


# ----------------------------------------------------------------------------- routed Q projection
@pytest.mark.parametrize("T,D,n_out,G,p", [(300, 512, 1024, 128, 0.5), (640, 1024, 2048, 512, 0.5),
                                           (200, 256, 1024, 256, 0.3), (1100, 512, 1536, 128, 0.7)])
def test_qproj_matches_oracle(ctx, T, D, n_out, G, p):
    from paper_2607_28418_b200 import binding
    rng = np.random.default_rng(T + G)
    x = synth.make_activations(rng, T, D, "bf16", "random")
    w = synth.make_weight(rng, n_out, D, 0.02, "bf16")
    mask = synth.bernoulli_mask(T, T, n_out // G, p)
    meta = meta_to_dev(wo.reorder(mask, 128))
    y = binding.wide_qproj(ctx, to_dev(x, "bf16"), to_dev(w, "bf16"), G, meta)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    ref = wo.qproj(x, w, mask, G)
    assert (y.float().cpu().numpy()[~wo.expand_group_mask(mask, G)] == 0.0).all()
    assert_close(y, ref, "qproj")


def test_qproj_closed_cases(ctx):
    from paper_2607_28418_b200 import binding
    T, D, n_out, G = 260, 256, 512, 128
    rng = np.random.default_rng(4)
    x = synth.make_activations(rng, T, D, "bf16", "random")
    w = synth.make_weight(rng, n_out, D, 0.02, "bf16")
    xd, wd = to_dev(x, "bf16"), to_dev(w, "bf16")
    ones = np.ones((T, n_out // G), dtype=bool)
    y = binding.wide_qproj(ctx, xd, wd, G, meta_to_dev(wo.reorder(ones, 128)))
    assert_close(y, x.astype(np.float64) @ w.astype(np.float64).T, "qproj dense")
    y0 = binding.wide_qproj(ctx, xd, wd, G, meta_to_dev(wo.reorder(~ones, 128)))
    assert (y0 == 0).all().item()
    with pytest.raises(binding.WideError):
        binding.wide_qproj(ctx, xd, wd, 64, meta_to_dev(wo.reorder(np.ones((T, n_out // 64), dtype=bool), 128)))


# ----------------------------------------------------------------------------- the attention half as a chain
def test_attention_half_chain_stage_by_stage(ctx):
    """route -> reorder -> routed Q projection -> masked attention -> O-projection on its already
    masked input.  Every stage is compared with the oracle applied to what the stage received."""
    from paper_2607_28418_b200 import binding
    from tests.gpu_util import bits_to_host
    T, D, H, hd, hpg = 640, 1024, 8, 128, 2
    NG, G = H // hpg, hpg * hd
    rng = np.random.default_rng(31)
    x = synth.make_activations(rng, T, D, "bf16", "random")
    w_r = synth.make_weight(rng, NG, D, 1.0 / np.sqrt(D), "bf16")
    w_q = synth.make_weight(rng, H * hd, D, 1.0 / np.sqrt(D), "bf16")     # unit-variance queries
    w_o = synth.make_weight(rng, D, H * hd, 0.02, "bf16")
    kv = synth.make_attn_case(32, T, T, H, H, hd)
    xd = to_dev(x, "bf16")
    bits, _ = binding.wide_route(ctx, xd, to_dev(w_r, "bf16"), NG, 2)
    mask = wo.mask_topk(wo.route_scores(x, w_r), 2)
    assert (bits_to_host(bits) == wo.pack_mask_bits(mask)).all()
    meta = binding.wide_reorder(ctx, bits, NG, 128)
    assert (meta["perm"].cpu().numpy() == wo.reorder(mask, 128)["perm"]).all()
    q = binding.wide_qproj(ctx, xd, to_dev(w_q, "bf16"), G, meta)
    assert_close(q, wo.qproj(x, w_q, mask, G), "chain: qproj")
    q_host = q.float().cpu().numpy()
    o = binding.wide_attn(ctx, q, to_dev(kv["k"].reshape(T, -1), "bf16"), to_dev(kv["v"].reshape(T, -1), "bf16"), H, H, hpg, meta)
    ref_o = wo.masked_attention(q_host.reshape(T, H, hd), kv["k"], kv["v"], mask, hpg)
    assert_close(o.reshape(T, H, hd), ref_o, "chain: attention")
    o_host = o.float().cpu().numpy()
    y = binding.wide_oproj(ctx, o, to_dev(w_o, "bf16"), G, bits, meta, flags=binding.FLAG_INPUT_MASKED)
    assert_close(y, wo.oproj(o_host, w_o, mask, G), "chain: oproj")
    torch.cuda.synchronize()
    assert ctx.status() == 0


# ----------------------------------------------------------------------------- decode form (split over the keys)
@pytest.mark.parametrize("t_q,t_k,h_q,h_kv,d,hpg", [
    (1, 1000, 8, 8, 128, 2),       # one new token, MHA
    (1, 4097, 32, 8, 128, 4),      # GQA 4:1, ragged key count
    (2, 300, 8, 2, 64, 4),         # two tokens, head_dim 64
    (4, 515, 4, 4, 128, 1),        # four tokens (speculative block), every head its own group
    (1, 17, 2, 2, 128, 1),         # fewer keys than one chunk
    (1, 20011, 8, 8, 128, 2),      # long cache: every warp goes round its ring stage several times
    (2, 9001, 8, 2, 64, 4),        # eight query rows per KV head, head_dim 64, many tiles
    (1, 40000, 8, 2, 128, 4),      # grouped-query decode, long cache: every warp reuses its stage several times
    (2, 30011, 8, 4, 64, 2),       # four rows per KV head, head_dim 64, long cache, ragged tail
])
@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("plain_loads", [False, True])
def test_attn_decode_matches_oracle(ctx, t_q, t_k, h_q, h_kv, d, hpg, causal, plain_loads):
    """Both decode kernels: K and V through the TMA ring (default) and by plain loads (WIDE_FLAG_SIMT)."""
    from paper_2607_28418_b200 import binding
    case = synth.make_attn_case(21, t_q, t_k, h_q, h_kv, d)
    mask = synth.bernoulli_mask(22 + t_k, t_q, h_q // hpg, 0.5)
    mask[0, 0] = True
    o = binding.wide_attn(ctx, to_dev(case["q"].reshape(t_q, -1), "bf16"), to_dev(case["k"].reshape(t_k, -1), "bf16"),
                          to_dev(case["v"].reshape(t_k, -1), "bf16"), h_q, h_kv, hpg, None, causal=causal,
                          mask_bits=bits_to_dev(wo.pack_mask_bits(mask)),
                          flags=binding.FLAG_SIMT if plain_loads else 0)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    ref = wo.masked_attention(case["q"], case["k"], case["v"], mask, hpg, causal=causal)
    got = o.reshape(t_q, h_q, d)
    assert (got.float().cpu().numpy()[~np.repeat(mask, hpg, axis=1)] == 0.0).all()
    assert_close(got, ref, "attn decode")


def test_attn_decode_and_prefill_forms_agree(ctx):
    from paper_2607_28418_b200 import binding
    t_q, t_k, h_q, h_kv, d, hpg = 2, 700, 8, 4, 128, 2
    case = synth.make_attn_case(23, t_q, t_k, h_q, h_kv, d)
    mask = synth.bernoulli_mask(24, t_q, h_q // hpg, 0.6)
    bits = bits_to_dev(wo.pack_mask_bits(mask))
    meta = meta_to_dev(wo.reorder(mask, 128))
    args = (to_dev(case["q"].reshape(t_q, -1), "bf16"), to_dev(case["k"].reshape(t_k, -1), "bf16"),
            to_dev(case["v"].reshape(t_k, -1), "bf16"), h_q, h_kv, hpg)
    a = binding.wide_attn(ctx, *args, meta, mask_bits=bits)                                    # decode form
    b = binding.wide_attn(ctx, *args, meta, mask_bits=bits, flags=binding.FLAG_FORCE_PREFILL)  # tcgen05 form
    ref = wo.masked_attention(case["q"], case["k"], case["v"], mask, hpg)
    assert_close(a.reshape(t_q, h_q, d), ref, "decode form")
    assert_close(b.reshape(t_q, h_q, d), ref, "prefill form")
    with pytest.raises(binding.WideError):
        binding.wide_attn(ctx, *args, None)                                                    # neither mask nor metadata
