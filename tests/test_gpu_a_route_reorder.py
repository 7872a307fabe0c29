"""GPU parity: wide_route, wide_reorder, wide_unpermute against the CPU oracle (bit-exact)."""
import os

import numpy as np
import pytest
import torch

from oracle import wide_oracle as wo
from paper_2607_28418_b200 import synth
from tests.gpu_util import bits_to_dev, bits_to_host, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_28418_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


def _route_case(cfg, seed, T):
    case = synth.make_ffn_case(cfg, seed, tokens=T)
    return case["x"], case["w_router"]


@pytest.mark.parametrize("dtype,T,D,NG,k", [("fp32", 128, 256, 16, 8), ("bf16", 300, 512, 86, 43),
                                            ("bf16", 1, 4096, 112, 56), ("bf16", 77, 1024, 224, 56),
                                            ("bf16", 64, 256, 33, 0), ("bf16", 64, 256, 33, 33)])
def test_route_topk_bit_exact(ctx, dtype, T, D, NG, k):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=T, hidden=D, d_ff=NG * 64, group=64, k=k, dtype=dtype)
    x, wr = _route_case(cfg, 5, T)
    ref = wo.pack_mask_bits(wo.mask_topk(wo.route_scores(x, wr), k))
    bits, scores = binding.wide_route(ctx, to_dev(x, dtype), to_dev(wr, dtype), NG, k, want_scores=True)
    assert (bits_to_host(bits) == ref).all()
    # the returned scores are diagnostics: fp32 tensor-core sums on the bf16 fast path
    tol = 1e-5 if dtype == "fp32" else 2e-3
    np.testing.assert_allclose(scores.cpu().numpy(), wo.route_scores(x, wr), rtol=tol, atol=tol)
    # the plain fp64 kernels must give the same bits
    bits2, _ = binding.wide_route(ctx, to_dev(x, dtype), to_dev(wr, dtype), NG, k, flags=binding.FLAG_SIMT)
    assert torch.equal(bits, bits2)


def test_route_fast_path_error_bound_and_near_ties(ctx):
    """Tensor-core scores stay inside the bound the guard band is built on, and rows that differ
    by one bf16 ulp in one weight (or not at all) are still ordered exactly."""
    from paper_2607_28418_b200 import binding
    T, D, NG, k = 512, 1024, 96, 48
    rng = np.random.default_rng(42)
    x = synth.round_to_bf16(rng.standard_normal((T, D)).astype(np.float32))
    base = synth.round_to_bf16((rng.standard_normal((1, D)) / np.sqrt(D)).astype(np.float32))
    wr = np.repeat(base, NG, axis=0)                     # all groups tie exactly ...
    for g in range(0, NG, 3):                            # ... except every third, off by one ulp somewhere
        i = int(rng.integers(0, D))
        wr[g, i] = synth.round_to_bf16(np.array([wr[g, i] * (1 + 2.0 ** -7)], dtype=np.float32))[0]
    wr = synth.round_to_bf16(wr)
    s_ref = wo.route_scores(x, wr)
    ref = wo.pack_mask_bits(wo.mask_topk(s_ref, k))
    bits, scores = binding.wide_route(ctx, to_dev(x, "bf16"), to_dev(wr, "bf16"), NG, k, want_scores=True)
    assert (bits_to_host(bits) == ref).all()
    eps = 2.0 ** -24 * D * np.linalg.norm(x, axis=1, keepdims=True) * np.linalg.norm(wr, axis=1).max()
    err = np.abs(scores.cpu().numpy().astype(np.float64) - s_ref)
    assert (err <= eps).all()
    assert err.max() <= 0.25 * eps.min()                 # measured error sits well inside the bound


def test_route_topk_ties_and_per_token_budget(ctx):
    from paper_2607_28418_b200 import binding
    T, D, NG = 40, 64, 20
    rng = np.random.default_rng(0)
    x = synth.round_to_bf16(rng.integers(-2, 3, size=(T, D)).astype(np.float32))   # many exact ties
    x[0] = 0.0
    wr = synth.round_to_bf16(rng.integers(-1, 2, size=(NG, D)).astype(np.float32))
    kt = rng.integers(0, NG + 1, size=T).astype(np.int32)
    ref = wo.pack_mask_bits(wo.mask_topk(wo.route_scores(x, wr), kt))
    bits, _ = binding.wide_route(ctx, to_dev(x, "bf16"), to_dev(wr, "bf16"), NG, 0,
                                 k_per_token=torch.from_numpy(kt).cuda())
    assert (bits_to_host(bits) == ref).all()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_route_pair_argmax_bit_exact(ctx, dtype):
    from paper_2607_28418_b200 import binding
    cfg = synth.CONFIGS["tiny"].with_(dtype=dtype)
    case = synth.make_ffn_case(cfg, 2)
    pr = synth.make_pair_router(cfg, 2, rank=16)
    logits = wo.route_logits_pair(case["x"], pr["w1"], pr["w2"])
    ref = wo.pack_mask_bits(wo.mask_pair_argmax(logits))
    bits, scores = binding.wide_route(ctx, to_dev(case["x"], dtype), to_dev(pr["w1"], dtype), cfg.n_groups,
                                      mode=binding.ROUTE_PAIR_ARGMAX, w2=to_dev(pr["w2"], dtype), rank=16,
                                      want_scores=True)
    assert (bits_to_host(bits) == ref).all()
    np.testing.assert_allclose(scores.cpu().numpy(), logits.reshape(cfg.tokens, -1), rtol=1e-5, atol=1e-5)


def test_route_pair_argmax_layer_size_and_near_ties(ctx):
    """The tensor-core form of Eq. 4 at a layer's size: pairs whose logits tie exactly, differ by one
    bf16 ulp of one weight, or differ only by rounding noise are all decided as fp64 decides them."""
    from paper_2607_28418_b200 import binding
    T, D, NG, rank = 1024, 2048, 86, 16
    rng = np.random.default_rng(11)
    x = synth.round_to_bf16(rng.standard_normal((T, D)).astype(np.float32))
    x[3] = 0.0                                                      # every pair ties
    w1 = synth.round_to_bf16((rng.standard_normal((D, rank)) / np.sqrt(D)).astype(np.float32))
    w2 = synth.round_to_bf16((rng.standard_normal((rank, NG, 2)) / np.sqrt(rank)).astype(np.float32))
    w2[:, 0::5, 1] = w2[:, 0::5, 0]                                 # exact ties for every token
    for g in range(1, NG, 5):                                       # one ulp apart in one row
        c = int(rng.integers(0, rank))
        w2[:, g, 1] = w2[:, g, 0]
        w2[c, g, 1] = synth.round_to_bf16(np.array([w2[c, g, 0] * (1 + 2.0 ** -7)], dtype=np.float32))[0]
    w2 = synth.round_to_bf16(w2).reshape(rank, 2 * NG)
    logits = wo.route_logits_pair(x, w1, w2)
    ref = wo.pack_mask_bits(wo.mask_pair_argmax(logits))
    xd, w1d, w2d = to_dev(x, "bf16"), to_dev(w1, "bf16"), to_dev(w2, "bf16")
    bits, scores = binding.wide_route(ctx, xd, w1d, NG, mode=binding.ROUTE_PAIR_ARGMAX, w2=w2d, rank=rank,
                                      want_scores=True)
    assert (bits_to_host(bits) == ref).all()
    np.testing.assert_allclose(scores.cpu().numpy(), logits.reshape(T, -1), rtol=2e-3, atol=2e-3)
    bits2, _ = binding.wide_route(ctx, xd, w1d, NG, mode=binding.ROUTE_PAIR_ARGMAX, w2=w2d, rank=rank,
                                  flags=binding.FLAG_SIMT)
    assert torch.equal(bits, bits2)


def test_route_pair_argmax_integer_ties(ctx):
    from paper_2607_28418_b200 import binding
    T, D, NG, rank = 256, 256, 40, 8
    rng = np.random.default_rng(3)
    x = synth.round_to_bf16(rng.integers(-2, 3, size=(T, D)).astype(np.float32))
    w1 = synth.round_to_bf16(rng.integers(-1, 2, size=(D, rank)).astype(np.float32))
    w2 = synth.round_to_bf16(rng.integers(-1, 2, size=(rank, 2 * NG)).astype(np.float32))
    ref = wo.pack_mask_bits(wo.mask_pair_argmax(wo.route_logits_pair(x, w1, w2)))
    bits, _ = binding.wide_route(ctx, to_dev(x, "bf16"), to_dev(w1, "bf16"), NG, mode=binding.ROUTE_PAIR_ARGMAX,
                                 w2=to_dev(w2, "bf16"), rank=rank)
    assert (bits_to_host(bits) == ref).all()


def test_route_argument_errors(ctx):
    from paper_2607_28418_b200 import binding
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.WideError) as e:
        binding.wide_route(ctx, x, w, 8, k=9)
    assert e.value.code == binding.ERR_INVALID_ARG
    with pytest.raises(binding.WideError) as e:
        binding.wide_route(ctx, x, torch.zeros((300, 64), dtype=torch.bfloat16, device="cuda"), 300, k=1)
    assert e.value.code == binding.ERR_UNSUPPORTED_SHAPE


# ----------------------------------------------------------------------------- reorder
def _check_reorder(ctx, mask, tile_m):
    from paper_2607_28418_b200 import binding
    T, NG = mask.shape
    ref = wo.reorder(mask, tile_m)
    out = binding.wide_reorder(ctx, bits_to_dev(wo.pack_mask_bits(mask)), NG, tile_m)
    torch.cuda.synchronize()
    assert (out["perm"].cpu().numpy() == ref["perm"]).all()
    assert (out["counts"].cpu().numpy() == ref["counts"]).all()
    assert (out["tile_map"].cpu().numpy() == ref["tile_map"]).all()
    nw = int(out["n_work"].item())
    assert nw == ref["n_work"]
    wl = out["work_list"].cpu().numpy()
    assert (wl[:nw] == ref["work_list"]).all() and (wl[nw:ref["tile_map"].size] == -1).all()
    nu = int(out["n_union"].item())
    assert nu == ref["n_union"]
    ul = out["union_list"].cpu().numpy()
    assert (ul[:nu] == ref["union_list"]).all() and (ul[nu:] == -1).all()
    assert (out["offsets"].cpu().numpy() == ref["offsets"]).all()
    assert (out["token_order"].cpu().numpy() == ref["token_order"]).all()
    assert (out["token_rank"].cpu().numpy() == ref["token_rank"]).all()
    return out, ref


def test_reorder_hand_worked_fixture(ctx):
    mask = np.array([[1, 0, 0], [0, 0, 1], [1, 0, 1], [0, 0, 0], [1, 0, 1], [1, 0, 0], [0, 0, 1]], dtype=bool)
    # tile_m must be a power of two >= 16 in the library; the fixture's tile_m = 3 is oracle-only,
    # so check the tile-independent outputs against the fixture text and the rest against the oracle
    out, _ = _check_reorder(ctx, mask, 16)
    assert out["perm"].cpu().numpy().tolist() == [[0, 2, 4, 5, 1, 3, 6], [0, 1, 2, 3, 4, 5, 6], [1, 2, 4, 6, 0, 3, 5]]
    assert out["counts"].cpu().numpy().tolist() == [4, 0, 4]


@pytest.mark.parametrize("T,NG,tile_m,p", [(1, 1, 128, 1.0), (1000, 86, 128, 0.5), (2048, 112, 128, 0.5),
                                           (777, 224, 64, 0.25), (513, 33, 16, 0.75), (300, 10, 128, 0.0),
                                           (300, 10, 128, 1.0), (4096, 256, 128, 0.5)])
def test_reorder_bit_exact(ctx, T, NG, tile_m, p):
    _check_reorder(ctx, synth.bernoulli_mask(T + NG, T, NG, p), tile_m)


def test_reorder_clusters_prototype_tokens(ctx):
    rng = np.random.default_rng(3)
    protos = rng.random((4, 112)) < 0.5
    which = rng.integers(0, 4, size=1500)
    out, ref = _check_reorder(ctx, protos[which], 128)
    order = out["token_order"].cpu().numpy()
    assert 1 + int((np.diff(which[order]) != 0).sum()) <= 5     # four runs (five if two keys collide)


def test_reorder_after_route_chain_and_determinism(ctx):
    from paper_2607_28418_b200 import binding
    cfg = synth.WideConfig("t", tokens=600, hidden=512, d_ff=86 * 64, group=64, k=43)
    case = synth.make_ffn_case(cfg, 9)
    bits, _ = binding.wide_route(ctx, to_dev(case["x"], "bf16"), to_dev(case["w_router"], "bf16"), 86, 43)
    a = binding.wide_reorder(ctx, bits, 86, 128)
    b = binding.wide_reorder(ctx, bits, 86, 128)
    for key in a:
        assert torch.equal(a[key], b[key])
    mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router"]), 43)
    ref = wo.reorder(mask, 128)
    assert (a["perm"].cpu().numpy() == ref["perm"]).all()
    assert int(a["counts"].sum().item()) == 600 * 43


# ----------------------------------------------------------------------------- unpermute
@pytest.mark.parametrize("dt", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("T,NG,G,p", [(300, 7, 64, 0.5), (129, 3, 128, 1.0), (64, 5, 8, 0.3)])
def test_unpermute_bit_exact(ctx, dt, T, NG, G, p):
    from paper_2607_28418_b200 import binding
    mask = synth.bernoulli_mask(T * 3 + NG, T, NG, p)
    ref_meta = wo.reorder(mask, 128)
    rng = np.random.default_rng(1)
    dense = synth.round_to_bf16(rng.standard_normal((T, NG * G)).astype(np.float32))
    packed = wo.gather_packed(dense, ref_meta["perm"], ref_meta["counts"], ref_meta["offsets"], G)
    if packed.shape[0] == 0:
        pytest.skip("nothing active")
    expect = wo.unpermute(packed, ref_meta["perm"], ref_meta["counts"], ref_meta["offsets"], T, G)
    meta = binding.wide_reorder(ctx, bits_to_dev(wo.pack_mask_bits(mask)), NG, 128)
    src = torch.from_numpy(packed).cuda().to(dt)
    dst = binding.wide_unpermute(ctx, src, meta, T, NG, G)
    assert (dst.float().cpu().numpy() == expect).all()
    if p == 1.0:
        assert (dst.float().cpu().numpy() == dense).all()   # gather then scatter = identity
